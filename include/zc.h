/*
 * zc.h — C ABI of the B200 lossless exponent / sign+mantissa Huffman codec.
 *
 * The library implements the data-parallel hot path of "Lossless Compression of
 * Neural Network Components: Weights, Checkpoints, and K/V Caches in
 * Low-Precision Formats" (Heilper & Singer, 2025): every BF16 / FP8 E4M3 /
 * FP4 E2M1 element is split into an exponent field and a sign+mantissa field
 * (Sec. 3.1, 3.2, 3.4), the fields of 1 / 2 / 4 neighbouring elements are
 * grouped into byte symbols (Fig. 7 caption for FP8 pairs; Sec. 3.4 for the 2-bit fields of four FP4
 * values that share a byte), each of the two symbol streams gets its own
 * Huffman code or is stored raw when it does not compress (Sec. 3.1), and the
 * result is written in fixed-size chunks that decode independently (Sec. 3.1:
 * chunks of fixed size with a little metadata each, so that any chunk can be
 * found and all chunks decode in parallel).  Decoding restores the original bit patterns exactly.
 *
 * Conventions
 *   - "d_" pointers are DEVICE pointers of the current CUDA device, "h_" pointers
 *     are HOST pointers.  The caller owns every buffer it passes.  The library
 *     owns plan and codebook objects until the matching *_destroy call.
 *   - `cuda_stream` is a cudaStream_t passed as void* (NULL = default stream).
 *     Device work is enqueued on it and is asynchronous unless stated otherwise.
 *   - The library allocates no device memory.  All device scratch is the
 *     caller's `d_workspace` of zc_workspace_bytes() bytes (256-byte aligned);
 *     its contents need not be initialised and are undefined afterwards.
 *     Two calls that overlap in time on the GPU must not share a workspace.
 *   - Device pointers d_in / d_out / d_comp / d_workspace must be 16-byte aligned.
 *   - Every function returns a zc_status; nothing throws; out-parameters are
 *     untouched on error.
 *
 * Geometry (fixed by the plan)
 *   G            elements per symbol: 1 (BF16), 2 (FP8), 4 (FP4)
 *   n_syms       ceil(n_elems / G) symbols in each of the two streams;
 *                stream 0 = exponent fields, stream 1 = sign+mantissa fields;
 *                element G*k+i sits in bits [w*i, w*i+w) of symbol k, w = 8/G;
 *                missing tail fields are zero
 *   chunk        chunk_bytes of element bytes = chunk_bytes/2 symbols per stream,
 *                cut into 32 equal subchunks
 *   code         canonical prefix code, lengths <= 12 bits, most significant bit
 *                first inside little-endian 32-bit words
 *
 * Container layout (little-endian; every section starts on a 16-byte boundary)
 *   header, 128 bytes
 *      0 u32 magic "ZC10"   4 u16 version = 1   6 u8 format   7 u8 n_streams = 2
 *      8 u64 n_elems       16 u32 chunk_bytes  20 u32 n_chunks
 *     24 u8 12 (max code length)  25 u8 G  26 u8 32 (subchunks)  27 u8 bytes per sub_end entry  28 u32 0
 *     32 u64 total_bytes   40 u64 payload_off  48 u64 payload_bytes  56 u64 0
 *     64 + 32 s : u8 mode (0 RAW, 1 HUFF), 7 zero bytes, u64 n_syms,
 *                 u64 payload_bits, u64 section_off            (s = 0, 1)
 *   one table section per HUFF stream (stream order):
 *      u8  code_len[256]            0 = symbol has no code
 *      u32 chunk_off16[n_chunks]    zero padded to a multiple of 16 bytes; offset of
 *                                   the chunk's bits from payload_off, in 16-byte units
 *      sub_end[n_chunks][32]        end bit of every subchunk inside its chunk; u16 entries when
 *                                   chunk_bytes <= 8192 (a chunk then holds < 65536 bits), else u32
 *   one body per RAW stream (stream order): n_syms symbol bytes, zero padded to 16
 *   payload area: for chunk 0, 1, ...: for each HUFF stream (stream order) the
 *      chunk's bits, zero padded to a multiple of 16 bytes
 *   16 zero guard bytes when at least one stream is HUFF
 *   Constant chunks: when both streams are HUFF, a chunk of a stream whose symbols are all the
 *      stream's fill symbol (the first symbol in (length, symbol) order, whose code is all zeros)
 *      has no payload at all: its 32 sub_end entries are 0, its piece is empty and its chunk_off16
 *      equals that of the piece that follows.  A chunk that holds symbols and has 0 bits can be
 *      nothing else.  This is what lets unchanged stretches of a delta checkpoint (Sec. 3.1, 4.1)
 *      cost less than the one bit per symbol of a per-symbol code.
 * The container is a pure function of (input bytes, plan, codebook).
 */
#ifndef ZC_H
#define ZC_H

#include <stddef.h>
#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

typedef enum zc_status {
    ZC_OK = 0,
    ZC_E_INVALID_ARG = 1,       /* null pointer, bad size, bad alignment, bad chunk size */
    ZC_E_UNSUPPORTED = 2,       /* unknown format or policy */
    ZC_E_BUFFER_TOO_SMALL = 3,  /* output capacity below zc_max_compressed_bytes() */
    ZC_E_CORRUPT = 4,           /* container does not match the plan or is damaged */
    ZC_E_CUDA = 5,              /* a CUDA runtime call failed */
    ZC_E_NOMEM = 6,             /* host allocation failed */
    ZC_E_DEVICE_TIMEOUT = 7,    /* a bounded wait inside a kernel gave up */
    ZC_E_NO_CODE = 8,           /* a symbol of the input has no code in the codebook */
    ZC_E_TOO_LARGE = 9          /* the tensor needs more built-in scratch than zc_compress_noalloc has */
} zc_status;

typedef enum zc_format {
    ZC_FMT_BF16 = 1,            /* u16 little-endian: sign 15, exponent 14..7, mantissa 6..0 */
    ZC_FMT_FP8_E4M3 = 2,        /* u8: sign 7, exponent 6..3, mantissa 2..0 */
    ZC_FMT_FP4_E2M1 = 3,        /* two per byte, element 2i in bits 3..0: sign 3, exponent 2..1, mantissa 0 */
    ZC_FMT_SCALE_U8 = 4,        /* a stream of scale bytes (E8M0 / E4M3 block scales of FP4 tensors, Sec. 3.4 and 4.4):
                                   one element per byte; the bytes at odd offsets are the symbols of stream 0, the
                                   bytes at even offsets those of stream 1 (a missing last odd byte counts as 0) */
    ZC_FMT_FP8_E5M2 = 5         /* u8: sign 7, exponent 6..2, mantissa 1..0 (Sec. 3.2).  Five exponent bits do not
                                   pair into byte symbols, so the coded field is the upper four exponent bits
                                   (bits 6..3); sign, lowest exponent bit and mantissa form the other field.
                                   Bit for bit the split of E4M3; the container records format 5 */
} zc_format;

typedef enum zc_policy {
    ZC_POLICY_AUTO = 0,         /* Huffman only for a stream that saves at least 1/64 (Sec. 3.1 rule) */
    ZC_POLICY_HUFF_ALL = 1,     /* Huffman for every non-empty stream */
    ZC_POLICY_RAW_ALL = 2,      /* both streams stored raw (split / merge only) */
    ZC_POLICY_STATIC = 3        /* a dictionary meant for OTHER tensors than the one it was counted on
                                   (Sec. 3.3, precomputed dictionaries): every one of the 256 symbols gets
                                   a code, so no later tensor can hit a missing code; the RAW / HUFF
                                   decision is the AUTO rule on the histogram given */
} zc_policy;

typedef enum zc_mode { ZC_MODE_RAW = 0, ZC_MODE_HUFF = 1 } zc_mode;

typedef struct zc_plan_s zc_plan_t;
typedef struct zc_codebook_s zc_codebook_t;
typedef struct zc_dict_s zc_dict_t;

typedef struct zc_dict_info {
    double tolerance;           /* as given to zc_dict_create */
    double baseline_ratio;      /* container bytes / input bytes of the first tensor coded since the last
                                   (re)build; 0 while there is none */
    double last_ratio;          /* of the latest observation; 0 before the first */
    uint64_t n_observed;        /* calls of zc_dict_observe */
    uint64_t n_rebuilds;        /* calls of zc_dict_rebuild */
    uint32_t has_baseline;
    uint32_t reserved;
} zc_dict_info;

typedef struct zc_plan_info {
    uint32_t format, group, chunk_bytes, n_chunks;
    uint64_t n_elems, n_syms, input_bytes;
    uint32_t syms_per_chunk, syms_per_subchunk;
} zc_plan_info;

typedef struct zc_stream_stats {
    uint64_t n_syms;            /* symbols in the stream */
    uint64_t raw_bits;          /* 8 * n_syms */
    uint64_t payload_bits;      /* sum count*len for HUFF, raw_bits for RAW */
    uint64_t container_bytes;   /* bytes this stream occupies in the container incl. its tables
                                   (0 when no header was given) */
    uint32_t mode;              /* zc_mode */
    uint32_t n_active_symbols;
    uint32_t max_len;
    uint32_t reserved;
    double avg_len;             /* sum count*len / n_syms with the codebook's lengths */
    double entropy_bits;        /* Shannon entropy of the histogram, bits per symbol */
} zc_stream_stats;

typedef struct zc_stats_t {
    zc_stream_stats stream[2];
    uint64_t in_bytes;          /* element bytes of the tensor */
    uint64_t out_bytes;         /* container bytes (header's total_bytes), 0 without header */
    double ratio_payload;       /* (payload_bits0 + payload_bits1) / (8 * in_bytes) */
    double ratio_container;     /* out_bytes / in_bytes, 0 without header */
} zc_stats_t;

/* ---- plan: problem statement of one tensor (Sec. 4: every tensor is compressed on its
 *      own, in chunks of one fixed size) -----------------------------------------------------
 * fmt         element format
 * n_elems     number of elements (0 is valid and gives a header-only container);
 *             must be even for FP4
 * chunk_bytes uncompressed element bytes per chunk: a multiple of 1024 in [1 KiB, ZC_MAX_CHUNK_BYTES]
 *             (64 KiB: what the kernels can hold of a chunk in shared memory with both streams coded;
 *             the container format itself has room for chunks of up to 256 KiB)
 * out         receives a new plan (host object; destroy with zc_plan_destroy)
 * Errors: INVALID_ARG (null out, bad chunk_bytes, odd FP4 count, more than 2^32-1 chunks),
 *         UNSUPPORTED (format), NOMEM. */
#define ZC_MAX_CHUNK_BYTES 65536u
zc_status zc_plan(zc_format fmt, uint64_t n_elems, uint32_t chunk_bytes, zc_plan_t** out);
void zc_plan_destroy(zc_plan_t* plan);
zc_status zc_plan_get_info(const zc_plan_t* plan, zc_plan_info* out);

/* Capacity in bytes that d_out of zc_compress must have: the size of the container when
 * every symbol of both streams takes a 12-bit code.  0 for a null plan. */
size_t zc_max_compressed_bytes(const zc_plan_t* plan);

/* Bytes of device scratch zc_compress / zc_decompress need.  0 for a null plan. */
size_t zc_workspace_bytes(const zc_plan_t* plan);

/* ---- split + histogram (Sec. 3.1-3.4 field split; the counts every Huffman code needs) ----
 * d_in    device, zc_plan_info.input_bytes bytes of elements
 * d_hist  device, uint64_t[2][256]; overwritten with the symbol counts of stream 0 and 1
 *         over the whole tensor (tail fields of a partial last symbol count as zero)
 * Asynchronous on cuda_stream.  Errors: INVALID_ARG, CUDA. */
zc_status zc_histogram(const zc_plan_t* plan, const void* d_in, uint64_t* d_hist, void* cuda_stream);

/* The histograms of many tensors with one call (one launch per 768 tensors).
 * plans    host array of n_tensors plans; all must have the same format
 * d_in     host array of DEVICE pointers (16-byte aligned), the tensors' element bytes
 * d_hists  device, uint64_t[n_tensors][2][256]; overwritten, d_hists[t] as by zc_histogram
 * Asynchronous on cuda_stream.  Errors: INVALID_ARG, CUDA. */
zc_status zc_histogram_batch(uint32_t n_tensors, const zc_plan_t* const* plans, const void* const* d_in,
                             uint64_t* d_hists, void* cuda_stream);

/* ---- codebook (Sec. 3.1 / 4.1: plain Huffman coding, one code per stream per tensor;
 *      Sec. 3.3 precomputed dictionaries: any histogram may be given) ------------------------
 * h_hist  host, uint64_t[2][256]
 * policy  which streams are Huffman-coded
 * out     receives a new codebook (host object, no device memory)
 * Lengths are those of an optimal prefix code with maximum length 12 (leaves ordered by
 * (count, symbol); leaf before package at equal weight); codes are canonical in
 * (length, symbol) order; a stream with one active symbol gets a 1-bit code.
 * Host-only: needs no GPU.  Errors: INVALID_ARG, UNSUPPORTED (policy), NOMEM. */
zc_status zc_build_codebook(const zc_plan_t* plan, const uint64_t* h_hist, zc_policy policy,
                            zc_codebook_t** out);
/* The codebooks of many tensors with one call, built on several host threads.
 * h_hists    host, uint64_t[n_tensors][2][256]
 * n_threads  host threads to use (0: as many as the machine has, at most 16, at least 8
 *            tensors per thread)
 * out        host array of n_tensors pointers; receives new codebooks, identical to those of
 *            zc_build_codebook; untouched on error
 * Errors: as zc_build_codebook. */
zc_status zc_build_codebooks(uint32_t n_tensors, const zc_plan_t* const* plans, const uint64_t* h_hists,
                             zc_policy policy, uint32_t n_threads, zc_codebook_t** out);
void zc_codebook_destroy(zc_codebook_t* cb);

/* Copy out one stream's mode, code lengths and right-aligned code values
 * (any of the three out pointers may be null). */
zc_status zc_codebook_get(const zc_codebook_t* cb, uint32_t stream, uint32_t* mode,
                          uint8_t* len256, uint32_t* code256);

/* ---- compress (Sec. 3.1 chunked entropy coding of both streams) ---------------------------
 * d_in          device, the tensor's element bytes
 * d_out         device, receives the container; out_capacity >= zc_max_compressed_bytes()
 * d_workspace   device scratch, zc_workspace_bytes() bytes
 * h_out_bytes   host, optional: when non-null the call synchronises cuda_stream, stores the
 *               container size and returns the device status (NO_CODE / DEVICE_TIMEOUT
 *               included); when null the call is asynchronous and the size is the
 *               header's total_bytes field
 * The codebook need not come from this tensor's histogram, but every symbol that occurs in
 * a HUFF stream must have a code; otherwise the device status becomes ZC_E_NO_CODE and the
 * container is invalid.
 * Errors: INVALID_ARG, BUFFER_TOO_SMALL, CUDA, and the device status when synchronous. */
zc_status zc_compress(const zc_plan_t* plan, const zc_codebook_t* cb, const void* d_in, void* d_out,
                      size_t out_capacity, void* d_workspace, uint64_t* h_out_bytes, void* cuda_stream);

/* ---- compress without a caller-supplied workspace ------------------------------------------
 * (No counterpart in the paper: an addition for callers that cannot allocate device memory.)
 *
 * Same operation and same result, byte for byte, as zc_compress, but the device scratch that
 * zc_compress takes as `d_workspace` lives inside the library: a fixed array in device memory
 * of ZC_NOALLOC_SCRATCH_BYTES bytes that every GPU loading the library holds until the process
 * exits.  It is meant for code that runs where cudaMalloc is off limits or unaffordable: inside
 * a memory pool that has handed out all of its budget, in a latency-critical serving loop that
 * must not touch the allocator, or in a plugin that is only given input and output buffers.
 * The call itself performs no cudaMalloc / cudaFree and calls no allocating library routine.
 *
 * d_in, d_out, out_capacity, h_out_bytes, cuda_stream: exactly as for zc_compress (the caller
 * still owns and passes input and output).
 *
 * Limit: the plan may have at most ZC_NOALLOC_MAX_CHUNKS chunks (n_chunks of zc_plan_info);
 * larger tensors are refused with ZC_E_TOO_LARGE and nothing is launched.  Use a larger
 * chunk_bytes, split the tensor, or call zc_compress with your own workspace.
 *
 * First call on a device: the library looks up the device address of its scratch array once
 * per device (with that device current) and remembers it.  Make that first call outside of
 * any stream capture.  Host threads may make it at the same time.  The remembered address
 * does not survive cudaDeviceReset: do not reset a device between calls.
 *
 * Asynchronous form (h_out_bytes == NULL): the caller holds no workspace pointer to read the
 * device status from (a symbol without code, a wait that gave up); zc_noalloc_status reads it
 * from the built-in array of the current device after waiting for the stream.
 *
 * Sharing: all calls on one device use the same scratch array.  Each call clears the part it
 * needs before use, so stale contents of an earlier call never matter, but two calls whose
 * GPU work overlaps in time (different streams, or different host threads) race on it and
 * corrupt each other's containers.  Serialise such calls on one stream.
 * Errors: as zc_compress, plus ZC_E_TOO_LARGE. */
#define ZC_NOALLOC_MAX_CHUNKS 65536u
#define ZC_NOALLOC_SCRATCH_BYTES (256u + 8u * ZC_NOALLOC_MAX_CHUNKS)
zc_status zc_compress_noalloc(const zc_plan_t* plan, const zc_codebook_t* cb, const void* d_in, void* d_out,
                              size_t out_capacity, uint64_t* h_out_bytes, void* cuda_stream);
/* Status word of the last zc_compress_noalloc call on the current device (waits for the stream):
 * ZC_OK, ZC_E_NO_CODE, ZC_E_DEVICE_TIMEOUT, or ZC_E_CUDA. */
zc_status zc_noalloc_status(void* cuda_stream);

/* ---- decompress (Sec. 3.1: chunks decode independently, in parallel) ------------------------
 * d_comp      device, a container made for the same plan; comp_bytes = bytes available
 * d_out       device, receives zc_plan_info.input_bytes bytes, identical to the original
 * The header is checked on the device against the plan before anything is decoded; a
 * mismatch or damaged table sets the device status to ZC_E_CORRUPT and nothing is written.
 * Asynchronous; read the outcome with zc_device_status().  Errors: INVALID_ARG, CUDA. */
zc_status zc_decompress(const zc_plan_t* plan, const void* d_comp, size_t comp_bytes, void* d_out,
                        void* d_workspace, void* cuda_stream);

/* ---- random access (Sec. 3.1: any chunk can be located and decoded on its own) ---------------
 * Decodes chunks first_chunk .. first_chunk + n_chunks - 1 of a container and nothing else.
 * d_out receives their element bytes, starting with the first byte of chunk first_chunk (so it
 * needs n_chunks * chunk_bytes bytes, fewer if the range includes the tensor's last chunk).
 * Everything else as zc_decompress (header and tables are checked the same way).
 * Errors: INVALID_ARG (also for a range that does not lie inside the plan's chunks), CUDA. */
zc_status zc_decompress_chunks(const zc_plan_t* plan, const void* d_comp, size_t comp_bytes,
                               uint32_t first_chunk, uint32_t n_chunks, void* d_out, void* d_workspace,
                               void* cuda_stream);

/* ---- compress many tensors with one call (Sec. 4 and 4.1: a model or a checkpoint is a set of
 *      tensors, each compressed on its own with its own codes; Sec. 3.3: K and V of all layers) -
 * The containers are byte for byte those of n_tensors calls of zc_compress; the chunks of all
 * tensors are handed out through one ticket counter, so that small tensors do not pay a launch
 * each (one launch per combination of stream modes that occurs and per 256 tensors of it).
 * n_tensors        number of tensors (0 returns ZC_OK and launches nothing)
 * plans            host array of n_tensors plans; all must have the same format and chunk_bytes
 * codebooks        host array, one codebook per tensor; tensors may share one (the pages of a K/V cache
 *                  coded with one dictionary): its tables are then uploaded once
 * d_in             host array of DEVICE pointers (16-byte aligned): the tensors' element bytes
 * d_out            host array of DEVICE pointers (16-byte aligned): d_out[t] receives container t
 * out_capacity     host array: out_capacity[t] >= zc_max_compressed_bytes(plans[t])
 * d_workspace      device scratch of workspace_bytes >= zc_compress_batch_workspace_bytes()
 *                  bytes (256-byte aligned); contents need not be initialised
 * h_out_bytes      host array of n_tensors sizes, optional: when non-null the call synchronises
 *                  cuda_stream, stores the container sizes and returns the device status; when
 *                  null the call is asynchronous (sizes are in the headers; status via
 *                  zc_batch_status)
 * The arrays are read before the call returns; the caller keeps ownership of everything.
 * (Large sets of code tables travel through a pinned host staging buffer that the library keeps
 * per calling thread; no device memory is allocated.)
 * Errors: INVALID_ARG (null or misaligned pointers, mixed formats or chunk sizes),
 * BUFFER_TOO_SMALL (an output or the workspace), UNSUPPORTED, CUDA, and the device status
 * (NO_CODE, DEVICE_TIMEOUT) when synchronous. */
size_t zc_compress_batch_workspace_bytes(uint32_t n_tensors, const zc_plan_t* const* plans);
zc_status zc_compress_batch(uint32_t n_tensors, const zc_plan_t* const* plans,
                            const zc_codebook_t* const* codebooks, const void* const* d_in,
                            void* const* d_out, const size_t* out_capacity, void* d_workspace,
                            size_t workspace_bytes, uint64_t* h_out_bytes, void* cuda_stream);

/* ---- decompress many tensors with one call (Sec. 4 and 4.1: a model or a checkpoint is a set of
 *      tensors, each compressed on its own; Sec. 3.3: the K and V tensors of all layers) --------
 * The result is the same as n_tensors calls of zc_decompress; the work of all tensors is spread
 * over the GPU in one launch (per 448 tensors), so that small tensors do not pay a launch and a
 * table build per block each.
 * n_tensors     number of tensors (0 returns ZC_OK and launches nothing)
 * plans         host array of n_tensors plans; all must have the same format and chunk_bytes
 * d_comp        host array of n_tensors DEVICE pointers (16-byte aligned), one container each
 * comp_bytes    host array: bytes available behind each d_comp[t]
 * d_out         host array of n_tensors DEVICE pointers (16-byte aligned); d_out[t] receives
 *               input_bytes of plans[t].  The outputs must not overlap.
 * d_workspace   device, at least 256 bytes (zc_workspace_bytes of any plan is enough)
 * The arrays are read before the call returns; the caller keeps ownership of everything.
 * A tensor whose header or tables are damaged is skipped (nothing of it is written), the others
 * are still decoded; the first error and its tensor are recorded on the device, read them with
 * zc_batch_status().  Asynchronous.
 * Errors: INVALID_ARG (null or misaligned pointers, mixed formats or chunk sizes), CORRUPT
 * (a comp_bytes[t] below the header size), UNSUPPORTED, CUDA. */
zc_status zc_decompress_batch(uint32_t n_tensors, const zc_plan_t* const* plans, const void* const* d_comp,
                              const size_t* comp_bytes, void* const* d_out, void* d_workspace,
                              void* cuda_stream);

/* Synchronise cuda_stream and return the status the last batch call on this workspace left on
 * the device (ZC_OK if none).  h_failed_tensor (optional, host) receives the index of the tensor
 * the first recorded error belongs to, or 0xFFFFFFFF. */
zc_status zc_batch_status(const void* d_workspace, uint32_t* h_failed_tensor, void* cuda_stream);

/* ---- XOR-delta forms (Sec. 3.1 and 4.1, delta checkpoints: the bitwise XOR of two consecutive
 *      checkpoints is what gets split and coded) ----------------------------------------------
 * Every call below is its namesake with one more argument, d_base: a DEVICE tensor of the same
 * size as the input (16-byte aligned; the batched calls take a host array of such pointers).
 * The XOR is fused into the kernels, nothing is materialised:
 *   zc_histogram_xor   counts the symbols of (d_in XOR d_base)
 *   zc_compress_xor    writes the container of (d_in XOR d_base)
 *   zc_decompress_xor  writes (decoded tensor XOR d_base), i.e. the tensor d_in was
 * A null d_base (for the batched calls: a null array, or a null entry) means "no base": the call
 * then is exactly its namesake.  The container does not record that it holds a delta: the
 * caller pairs it with the right base.  Errors: as the namesakes. */
zc_status zc_histogram_xor(const zc_plan_t* plan, const void* d_in, const void* d_base, uint64_t* d_hist,
                           void* cuda_stream);
zc_status zc_histogram_batch_xor(uint32_t n_tensors, const zc_plan_t* const* plans, const void* const* d_in,
                                 const void* const* d_base, uint64_t* d_hists, void* cuda_stream);
zc_status zc_compress_xor(const zc_plan_t* plan, const zc_codebook_t* cb, const void* d_in, const void* d_base,
                          void* d_out, size_t out_capacity, void* d_workspace, uint64_t* h_out_bytes,
                          void* cuda_stream);
zc_status zc_compress_batch_xor(uint32_t n_tensors, const zc_plan_t* const* plans,
                                const zc_codebook_t* const* codebooks, const void* const* d_in,
                                const void* const* d_base, void* const* d_out, const size_t* out_capacity,
                                void* d_workspace, size_t workspace_bytes, uint64_t* h_out_bytes,
                                void* cuda_stream);
zc_status zc_decompress_xor(const zc_plan_t* plan, const void* d_comp, size_t comp_bytes, const void* d_base,
                            void* d_out, void* d_workspace, void* cuda_stream);
zc_status zc_decompress_batch_xor(uint32_t n_tensors, const zc_plan_t* const* plans, const void* const* d_comp,
                                  const size_t* comp_bytes, const void* const* d_base, void* const* d_out,
                                  void* d_workspace, void* cuda_stream);

/* Synchronise cuda_stream and return the status word the last zc_compress / zc_decompress
 * call on this workspace left on the device (ZC_OK if none was raised). */
zc_status zc_device_status(const zc_plan_t* plan, const void* d_workspace, void* cuda_stream);

/* ---- host-side checks and statistics ------------------------------------------------------
 * zc_validate_container: structural check of a HOST copy of a container against a plan:
 * header fields, section bounds, Kraft sum of each code-length table, monotone chunk
 * offsets and subchunk ends, payload bit totals.  Returns ZC_OK or ZC_E_CORRUPT. */
zc_status zc_validate_container(const zc_plan_t* plan, const void* h_container, size_t bytes);

/* zc_stats (Sec. 4 reports exponent and mantissa results separately): per-stream and total
 * sizes and ratios from a histogram and a codebook; h_header (host copy of at least the first
 * 128 container bytes) is optional and adds the container-inclusive figures. */
zc_status zc_stats(const zc_plan_t* plan, const zc_codebook_t* cb, const uint64_t* h_hist,
                   const void* h_header, zc_stats_t* out);

/* ---- runtime dictionaries for K/V cache tensors (Sec. 3.3: dictionaries are computed ahead of
 *      time while the exponent distribution stays stable, and replaced only when the achieved
 *      ratio gets worse; Sec. 5.2 reports the savings of such static dictionaries) -------------
 * A zc_dict_t owns one ZC_POLICY_STATIC codebook and the bookkeeping that decides when to replace
 * it.  The paper gives no threshold; here the caller does: `tolerance` is the relative growth of
 * the container ratio (container bytes / input bytes) over the baseline that is still accepted.
 * The baseline is the ratio of the first tensor observed after the dictionary was (re)built.
 * Host-only objects; one dictionary per kind of tensor (say, per layer and K or V), used from
 * one thread at a time.
 *
 * zc_dict_create   codebook from the histogram of a representative tensor (h_hist as for
 *                  zc_build_codebook); tolerance >= 0.  Errors: INVALID_ARG, NOMEM.
 * zc_dict_codebook the current codebook, for zc_compress / zc_compress_batch on tensors of the
 *                  same format; owned by the dictionary, valid until zc_dict_rebuild / destroy.
 * zc_dict_observe  report one coded tensor: input_bytes > 0 and the container size the compress
 *                  call returned.  *rebuild is set to 1 when container_bytes / input_bytes exceeds
 *                  baseline * (1 + tolerance), else 0; the first observation after a (re)build
 *                  becomes the baseline and never asks for a rebuild.  Errors: INVALID_ARG.
 * zc_dict_rebuild  replace the codebook by one built from h_hist (the histogram of the tensor
 *                  that was coded badly); the baseline is taken anew from the next observation.
 *                  The caller compresses that tensor again if it wants the better ratio now.
 * zc_dict_get_info the bookkeeping above. */
zc_status zc_dict_create(const zc_plan_t* plan, const uint64_t* h_hist, double tolerance, zc_dict_t** out);
void zc_dict_destroy(zc_dict_t* dict);
const zc_codebook_t* zc_dict_codebook(const zc_dict_t* dict);
zc_status zc_dict_observe(zc_dict_t* dict, uint64_t input_bytes, uint64_t container_bytes, int* rebuild);
zc_status zc_dict_rebuild(zc_dict_t* dict, const zc_plan_t* plan, const uint64_t* h_hist);
zc_status zc_dict_get_info(const zc_dict_t* dict, zc_dict_info* out);

const char* zc_strerror(zc_status s);

#ifdef __cplusplus
}
#endif
#endif /* ZC_H */
