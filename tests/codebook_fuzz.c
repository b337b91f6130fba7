/* Test program: the library's codebook builder against the oracle's on many generated histograms.
 *
 *   codebook_fuzz <libzc.so> <libzc_oracle.so> <n_histograms> <seed>
 *
 * Both libraries are opened with dlopen, so this file shares no code with either.  Each round builds one
 * codebook (two histograms, one per stream) with zc_build_codebook and compares code lengths, code values and
 * stream modes with zo_code_lengths / zo_static_lengths, zo_canonical_codes and zo_choose_mode.  The histogram
 * kinds cover what a length-limited builder gets wrong first: ties everywhere (all counts equal, counts from a
 * set of two or three values), Fibonacci and power-of-two profiles (unlimited Huffman depth far above 12),
 * counts around 2^33 (sums beyond 32 bits), geometric tails, few active symbols, and plain random counts.
 * Prints "ok <n>" and exits 0, or prints the first difference and exits 1.
 */
#include <dlfcn.h>
#include <stdint.h>
#include <stdio.h>
#include <stdlib.h>
#include <string.h>

typedef struct zc_plan zc_plan_t;
typedef struct zc_codebook zc_codebook_t;
typedef int (*zc_plan_create_fn)(int, uint64_t, uint32_t, zc_plan_t**);
typedef void (*zc_plan_destroy_fn)(zc_plan_t*);
typedef int (*zc_build_codebook_fn)(const zc_plan_t*, const uint64_t*, int, zc_codebook_t**);
typedef void (*zc_codebook_destroy_fn)(zc_codebook_t*);
typedef int (*zc_codebook_get_fn)(const zc_codebook_t*, uint32_t, uint32_t*, uint8_t*, uint32_t*);
typedef int (*zo_lengths_fn)(const uint64_t*, int, uint8_t*);
typedef void (*zo_codes_fn)(const uint8_t*, uint32_t*);
typedef int (*zo_mode_fn)(const uint64_t*, const uint8_t*, int);

static uint64_t rng_state;
static uint64_t rnd(void)  /* splitmix64 */
{
    uint64_t z = (rng_state += 0x9E3779B97F4A7C15ull);
    z = (z ^ (z >> 30)) * 0xBF58476D1CE4E5B9ull;
    z = (z ^ (z >> 27)) * 0x94D049BB133111EBull;
    return z ^ (z >> 31);
}
static uint64_t below(uint64_t n) { return n ? rnd() % n : 0; }

static void make_histogram(uint64_t h[256], uint64_t round)
{
    uint64_t c[256];
    int kind = (int)(round % 10);
    int n = (round % 3 == 0) ? (int)below(12) : (int)below(257);
    if (round % 97 == 0) n = 256;
    uint64_t a = 1, b = 1;
    uint64_t base = 1 + below(1u << 20);
    double decay = 0.05 + (double)below(1000) / 1000.0;
    double g = 1e7;
    for (int i = 0; i < n; ++i) {
        switch (kind) {
        case 0: c[i] = base; break;                                          /* all equal */
        case 1: c[i] = 1 + below(3); break;                                  /* ties among few values */
        case 2: c[i] = a; { uint64_t t = a + b; a = b; b = t < (1ull << 40) ? t : (1ull << 40); } break; /* Fibonacci */
        case 3: c[i] = 1ull << (i < 40 ? i : 40); break;                     /* powers of two */
        case 4: c[i] = (1ull << 33) - 5 + below(10); break;                  /* around 2^33 */
        case 5: c[i] = (uint64_t)g + 1; g *= (1.0 - decay * 0.6); break;     /* geometric tail: the limit binds */
        case 6: c[i] = 1ull << below(30); break;                             /* random powers of two */
        case 7: c[i] = 1 + below(1u << 30); break;                           /* random */
        case 8: c[i] = 1 + below(1000) * below(1000); break;                 /* products, many small */
        default: c[i] = (i % 7 == 0) ? (1ull << 33) + below(3) : 1 + below(4); break; /* giants among dwarfs */
        }
    }
    /* scatter over the symbol values (a partial Fisher-Yates shuffle of the positions) */
    uint8_t pos[256];
    for (int i = 0; i < 256; ++i) pos[i] = (uint8_t)i;
    int scatter = (round / 10) % 2;
    for (int i = 0; i < 256; ++i) h[i] = 0;
    for (int i = 0; i < n; ++i) {
        int j = scatter ? i + (int)below((uint64_t)(256 - i)) : i;
        uint8_t t = pos[i]; pos[i] = pos[j]; pos[j] = t;
        h[pos[i]] = c[i];
    }
}

#define SYM(lib, name) dlsym(lib, name)

int main(int argc, char** argv)
{
    if (argc != 5) { fprintf(stderr, "usage: %s libzc libzo n seed\n", argv[0]); return 2; }
    void* zc = dlopen(argv[1], RTLD_NOW | RTLD_LOCAL);
    void* zo = dlopen(argv[2], RTLD_NOW | RTLD_LOCAL);
    if (!zc || !zo) { fprintf(stderr, "dlopen: %s\n", dlerror()); return 2; }
    uint64_t n = strtoull(argv[3], 0, 10);
    rng_state = strtoull(argv[4], 0, 10);
    zc_plan_create_fn plan_create = (zc_plan_create_fn)SYM(zc, "zc_plan");
    zc_plan_destroy_fn plan_destroy = (zc_plan_destroy_fn)SYM(zc, "zc_plan_destroy");
    zc_build_codebook_fn build = (zc_build_codebook_fn)SYM(zc, "zc_build_codebook");
    zc_codebook_destroy_fn cb_destroy = (zc_codebook_destroy_fn)SYM(zc, "zc_codebook_destroy");
    zc_codebook_get_fn cb_get = (zc_codebook_get_fn)SYM(zc, "zc_codebook_get");
    zo_lengths_fn zo_lengths = (zo_lengths_fn)SYM(zo, "zo_code_lengths");
    zo_lengths_fn zo_static = (zo_lengths_fn)SYM(zo, "zo_static_lengths");
    zo_codes_fn zo_codes = (zo_codes_fn)SYM(zo, "zo_canonical_codes");
    zo_mode_fn zo_mode = (zo_mode_fn)SYM(zo, "zo_choose_mode");
    if (!plan_create || !plan_destroy || !build || !cb_destroy || !cb_get || !zo_lengths || !zo_static || !zo_codes || !zo_mode) {
        fprintf(stderr, "missing symbol\n");
        return 2;
    }
    zc_plan_t* plan = 0;
    if (plan_create(1 /* BF16 */, 16, 1024, &plan) != 0) { fprintf(stderr, "plan\n"); return 2; }

    uint64_t h[2][256];
    uint64_t done = 0;
    for (uint64_t round = 0; done < n; ++round) {
        make_histogram(h[0], round);
        make_histogram(h[1], round * 7 + 3);
        int policy = (round % 4 == 3) ? 3 /* STATIC */ : (round % 4 == 2) ? 1 /* HUFF_ALL */ : 0 /* AUTO */;
        zc_codebook_t* cb = 0;
        int rc = build(plan, &h[0][0], policy, &cb);
        if (rc != 0) { printf("round %llu: zc_build_codebook returned %d\n", (unsigned long long)round, rc); return 1; }
        for (uint32_t s = 0; s < 2; ++s) {
            uint32_t mode = 99, code[256], want_code[256];
            uint8_t len[256], want_len[256];
            cb_get(cb, s, &mode, len, code);
            memset(want_len, 0, sizeof want_len);
            int orc = (policy == 3 ? zo_static : zo_lengths)(h[s], 12, want_len);
            if (orc != 0) { printf("round %llu: oracle lengths returned %d\n", (unsigned long long)round, orc); return 1; }
            zo_codes(want_len, want_code);
            int want_mode = zo_mode(h[s], want_len, policy);
            if (memcmp(len, want_len, 256) || memcmp(code, want_code, sizeof code) || (int)mode != want_mode) {
                printf("round %llu stream %u policy %d: differs (mode %u want %d)\n", (unsigned long long)round, s, policy, mode, want_mode);
                for (int i = 0; i < 256; ++i)
                    if (h[s][i]) printf("  sym %d count %llu len %u want %u\n", i, (unsigned long long)h[s][i], len[i], want_len[i]);
                return 1;
            }
            ++done;
        }
        cb_destroy(cb);
    }
    plan_destroy(plan);
    printf("ok %llu\n", (unsigned long long)done);
    return 0;
}
