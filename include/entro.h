/*
 * entro.h -- C ABI of the B200 (sm_100a) library for EntroLLM's weight path:
 * per-tensor quantisation, symbol histogram, canonical Huffman codebook, encoding into a
 * bitstream with a per-chunk bit-offset index, and parallel decoding fused with
 * dequantisation to fp16.
 *
 * General rules
 *  - Pointers named *_dev are CUDA device pointers on the current device; pointers named
 *    *_host are host pointers.  The caller owns and allocates every buffer it passes.
 *    The library keeps a small per-device workspace of its own (decode tables, work
 *    descriptors, a status word), allocated on first use and grown on demand.
 *  - cuda_stream is a cudaStream_t passed as void* (NULL = the default stream).
 *  - Every call returns an entro_status.  Nothing throws, aborts or traps.  Argument
 *    errors are found before any kernel is launched.
 *  - Calls that return data to the host (qp_host, counts_host, total_bits_host)
 *    synchronise cuda_stream before returning.  Decode calls are asynchronous.
 *  - Symbols are one per byte (values 0 .. 2^bits - 1), bits is 4 or 8.
 *  - Calls on one device share the workspace: issue them on one stream, or order them
 *    with events, so that no two of them overlap on the GPU.  Host-side entry is
 *    serialised by an internal lock.
 *
 * Compressed format (fixed here; the paper leaves it open)
 *  - Stream: 32-bit words; stream bit i is bit (31 - i % 32) of word i / 32; a codeword is
 *    written MSB-first, codewords follow one another without gaps in the order given below;
 *    unused bits are zero.  A stream buffer holds ceil(total_bits / 32) +
 *    ENTRO_STREAM_SLACK_WORDS words, the slack zero, and starts on a 16-byte boundary.
 *  - Segments: the paper decodes independent segments with known boundaries in parallel
 *    (Section 3, "Segmentation for parallel Huffman decoding"; Fig. 3).  Here a segment is
 *    a chunk of chunk_symbols consecutive symbols of one tensor in row-major element order
 *    (the last chunk may be short); the chunks' bits follow one another in the stream.
 *  - Order inside a chunk (the paper fixes the boundaries, not this).  The chunk's m symbols
 *    e[0 .. m) form groups of 8 consecutive symbols: group g = e[8 g .. 8 g + 8) (the last
 *    group is short if m is not a multiple of 8).  Group g belongs to sub-block g mod 32.
 *    The stream holds sub-block 0 first, then sub-block 1, ... sub-block 31; a sub-block
 *    holds its groups in ascending g (l, l + 32, l + 64, ...), and a group its symbols in
 *    element order.  A sub-block without a group (short last chunk) is empty.  So the
 *    stored order of a full chunk of 4096 symbols starts e[0..8), e[256..264), e[512..520),
 *    ..., e[3840..3848), then sub-block 1: e[8..16), e[264..272), ...
 *    (32 decoder lanes can then start inside a chunk without searching, and what they decode
 *    in one step is contiguous in the output.)
 *  - Index of a tensor with n_chunks = ceil(n / chunk_symbols) chunks:
 *        uint64_t offsets[n_chunks + 1];      stream bit at which each chunk starts,
 *                                             offsets[n_chunks] = total bits
 *        uint16_t sub_len[n_chunks][32];      bits of sub-block l of chunk c (0 if empty);
 *                                             the 32 values of a chunk sum to
 *                                             offsets[c + 1] - offsets[c]
 *    stored back to back (entro_index_bytes bytes), 8-byte aligned.
 *  - chunk_symbols is a multiple of 32, at least 32 and at most 16384.
 */
#ifndef ENTRO_H
#define ENTRO_H

#include <stdint.h>

#ifdef __cplusplus
extern "C" {
#endif

#define ENTRO_MAX_SYMBOLS 256
#define ENTRO_MAX_CODE_LEN 32
#define ENTRO_SUB_BLOCKS 32
#define ENTRO_STREAM_SLACK_WORDS 8
#define ENTRO_MAX_CHUNK_SYMBOLS 16384
#define ENTRO_STATIC_MAX_TENSORS 8
#define ENTRO_GEMV_MAX_BATCH 8

typedef enum {
    ENTRO_OK = 0,
    ENTRO_ERR_INVALID_ARG = 1,
    ENTRO_ERR_BUFFER_TOO_SMALL = 2,
    ENTRO_ERR_NONFINITE = 3,       /* the tensor holds a NaN or an infinity */
    ENTRO_ERR_CODE_TOO_LONG = 4,   /* an optimal code length exceeds 32 bits */
    ENTRO_ERR_CORRUPT_STREAM = 5,  /* stream, index and codebook do not agree */
    ENTRO_ERR_CUDA = 6,            /* a CUDA runtime call failed */
    ENTRO_ERR_UNSUPPORTED = 7,
    ENTRO_ERR_TOO_MANY_TENSORS = 8 /* more tensors than entro_decode_dequant_static has room for */
} entro_status;

/* Every tensor is quantised in one of two modes, unsigned or asymmetric, chosen from its
 * weight distribution (Section 3, "Mixed Quantization Scheme", Eq. 1).  The paper does not
 * give the rule; AUTO: unsigned iff every weight is >= 0. */
typedef enum { ENTRO_MODE_AUTO = 0, ENTRO_MODE_UNSIGNED = 1, ENTRO_MODE_ASYMMETRIC = 2 } entro_mode;

typedef struct {
    int32_t bits;        /* 4 or 8 */
    int32_t mode;        /* resolved: ENTRO_MODE_UNSIGNED or ENTRO_MODE_ASYMMETRIC */
    float scale;         /* s */
    int32_t zero_point;  /* z, an integer in [0, 2^bits - 1]; 0 in unsigned mode */
    float lo, hi;        /* tensor minimum and maximum */
} entro_qparams;

typedef struct {
    int32_t nsym;                       /* alphabet size, 1 .. 256 */
    int32_t max_len;                    /* longest code length in use */
    uint8_t len[ENTRO_MAX_SYMBOLS];     /* code length per symbol, 0 = symbol unused */
    uint32_t code[ENTRO_MAX_SYMBOLS];   /* canonical code, right-aligned in len bits */
} entro_codebook;

/* One compressed tensor for the batched decode.  Host struct; the pointers inside are
 * device pointers. */
typedef struct {
    const uint32_t *stream_dev;   /* 16-byte aligned */
    uint64_t stream_words;        /* words in the buffer, slack included */
    const void *index_dev;        /* 8-byte aligned, entro_index_bytes(n, chunk_symbols) bytes */
    uint64_t n;                   /* symbols (= weights) in the tensor */
    uint32_t chunk_symbols;
    float scale;
    int32_t zero_point;
    entro_codebook cb;            /* only nsym and len[] are read by the decoder */
    void *out_fp16_dev;           /* n fp16 values, 16-byte aligned */
} entro_tensor_desc;

/*
 * Quantise one tensor (Section 3, "Mixed Quantization Scheme", Eq. 1).
 *   lo, hi = min, max of the weights.  qmax = 2^bits - 1.
 *   unsigned:   s = hi / qmax, z = 0.
 *   asymmetric: s = (hi - lo) / qmax, z = clamp(rne(-lo / s), 0, qmax).
 *   q = clamp(rne(w / s) + z, 0, qmax), so that w_hat = s * (q - z).
 * All arithmetic is IEEE fp32 with true division; rne is round-half-to-even.  If the
 * computed s is not positive (constant tensor), s = 1.
 * w_fp16_dev: n fp16 weights (device, 16-byte aligned).  q_dev: n bytes (device, 16-byte
 * aligned), one symbol per byte.  qp_host: filled on return.  Synchronises.
 * ENTRO_ERR_NONFINITE if a weight is NaN or infinite (q_dev is then not written).
 */
entro_status entro_quantize_tensor(const void *w_fp16_dev, uint64_t n, int bits, entro_mode mode,
                                   uint8_t *q_dev, entro_qparams *qp_host, void *cuda_stream);

/*
 * The grid the paper argues against, for comparison (Section 3, "Mixed Quantization
 * Scheme"; Table 2, column "SOTA"): block-based quantisation.  Every run of `block`
 * consecutive weights (the paper's example is 32; the last run may be shorter) gets a range,
 * mode, s and z of its own by the rules of entro_quantize_tensor, and is quantised with
 * them.  The paper's point is that such grids flatten the histogram of the codes, so that
 * entropy coding saves little; entro_histogram and entro_build_codebook on q_dev measure it.
 * w_fp16_dev: n fp16 weights (device).  q_dev: n bytes (device), one symbol per byte.
 * scales_dev / zero_points_dev: ceil(n / block) values each (device), or NULL if not wanted.
 * Synchronises.  ENTRO_ERR_NONFINITE if a weight is NaN or infinite (blocks that hold one
 * are left unwritten).
 */
entro_status entro_quantize_blocks(const void *w_fp16_dev, uint64_t n, int bits, entro_mode mode,
                                   uint32_t block, uint8_t *q_dev, float *scales_dev,
                                   int32_t *zero_points_dev, void *cuda_stream);

/*
 * Symbol frequencies, the "score" each symbol gets in Section 3 ("Huffman weight
 * encoding").  counts_host[k] = number of symbols equal to k, k < 2^bits.  Synchronises.
 * ENTRO_ERR_INVALID_ARG if a symbol is >= 2^bits.
 */
entro_status entro_histogram(const uint8_t *q_dev, uint64_t n, int bits, uint64_t *counts_host,
                             void *cuda_stream);

/*
 * Huffman code lengths by recursive merging of the two least frequent nodes (Section 3,
 * "Huffman weight encoding"), then canonical codes.  Pure host code.
 * Ties: on equal weight a leaf is taken before an internal node, leaves by ascending
 * symbol, internal nodes by creation order.  Symbols with count 0 get length 0; a single
 * used symbol gets length 1, code 0.  Canonical codes: symbols ordered by (length,
 * symbol), the first code is 0, each next code is (previous + 1) << (growth in length).
 * ENTRO_ERR_CODE_TOO_LONG if a length exceeds 32; ENTRO_ERR_INVALID_ARG if all counts
 * are zero or nsym is outside 1 .. 256.
 */
entro_status entro_build_codebook(const uint64_t *counts_host, int nsym, entro_codebook *cb_host);

/*
 * The same with a cap on the code length: the cheapest prefix code none of whose codes is
 * longer than max_len (package-merge), then canonical codes.  NOT the paper's code: Section 3
 * uses the unrestricted Huffman code, which no prefix code beats; a capped code costs more
 * (measured on the benchmark's 8-bit weights: +0.045 bit per weight at max_len = 12, +0.18
 * at 10; nothing at 4 bits) and bounds the decoder's table depth.  An optional variant of
 * the format; streams made with it decode with the ordinary decode calls, somewhat more
 * slowly than Huffman streams: this library's tables are shaped for codes that grow long
 * towards the all-ones end, which a capped code does less.  Steps (fixed so that
 * the result is unique): leaves ascending by (count, symbol); for level j = max_len .. 1 the
 * list is the leaves merged with the packages of level j + 1, ascending by weight, a leaf
 * before a package of equal weight, packages in the order they were made; packages are the
 * consecutive pairs of a list; a symbol's length is the number of the first 2 (n - 1) items
 * of level 1 that contain it.  ENTRO_ERR_CODE_TOO_LONG if 2^max_len is less than the number
 * of used symbols; ENTRO_ERR_INVALID_ARG for max_len outside 1 .. 32.
 */
entro_status entro_build_codebook_limited(const uint64_t *counts_host, int nsym, int max_len,
                                          entro_codebook *cb_host);

/* Words a stream buffer needs for these counts under this codebook: ceil(sum count[k] *
 * len[k] / 32) + ENTRO_STREAM_SLACK_WORDS.  0 on a bad argument. */
uint64_t entro_stream_words(const uint64_t *counts_host, const entro_codebook *cb_host);

/* Upper bound of the same without a histogram: n symbols of max_len bits each. */
uint64_t entro_encode_bound_words(uint64_t n, const entro_codebook *cb_host);

/* Bytes of the index of an n-symbol tensor: 8 * (n_chunks + 1) + 64 * n_chunks. */
uint64_t entro_index_bytes(uint64_t n, uint32_t chunk_symbols);

/*
 * Encode symbols into the compressed format described at the top (Section 3: variable
 * length codes, segments with known boundaries).  q_dev: n symbols, one per byte (device,
 * 16-byte aligned).  stream_dev (16-byte aligned,
 * stream_cap_words words) is zeroed and filled; index_dev (8-byte aligned) receives the
 * offsets and sub-block lengths; *total_bits_host the stream length in bits.  Synchronises.
 * ENTRO_ERR_BUFFER_TOO_SMALL if the stream needs more than stream_cap_words -
 * ENTRO_STREAM_SLACK_WORDS words or the index more than index_cap_bytes;
 * ENTRO_ERR_INVALID_ARG if a symbol has no code or a buffer is not aligned as stated.
 */
entro_status entro_encode(const uint8_t *q_dev, uint64_t n, const entro_codebook *cb_host,
                          uint32_t chunk_symbols, uint32_t *stream_dev, uint64_t stream_cap_words,
                          void *index_dev, uint64_t index_cap_bytes, uint64_t *total_bits_host,
                          void *cuda_stream);

/*
 * The offline stages for many tensors with one synchronisation per stage instead of several
 * per tensor (a whole model is compressed in a fraction of a second).  Results are those of
 * the per-tensor calls, bit for bit.
 *
 * entro_quantize_histogram_batched: for every job, the range of the tensor, (s, z) from it
 * (computed on the device with the arithmetic stated at entro_quantize_tensor), the symbols
 * q_dev, and their frequencies, counted in the pass that writes them.  qp_host[j] and
 * counts_host[j * ENTRO_MAX_SYMBOLS .. + 2^bits) are filled on return (counts beyond 2^bits
 * are 0).  ENTRO_ERR_NONFINITE if a tensor holds a NaN or an infinity (that tensor's q_dev is
 * not written, its counts are 0; the other tensors are complete).
 *
 * entro_encode_batched: entro_encode for every job; total_bits_host[j] on return.
 * ENTRO_ERR_BUFFER_TOO_SMALL if a stream does not fit its buffer (that stream is left
 * zeroed), ENTRO_ERR_INVALID_ARG if a symbol has no code; the other tensors are complete.
 */
typedef struct {
    const void *w_fp16_dev;   /* n fp16 weights, 16-byte aligned */
    uint64_t n;
    int32_t bits;             /* 4 or 8 */
    int32_t mode;             /* entro_mode */
    uint8_t *q_dev;           /* n bytes, 16-byte aligned */
} entro_quantize_job;

typedef struct {
    const uint8_t *q_dev;     /* n symbols, 16-byte aligned */
    uint64_t n;
    const entro_codebook *cb_host;
    uint32_t chunk_symbols;
    uint32_t reserved;        /* 0 */
    uint32_t *stream_dev;     /* 16-byte aligned */
    uint64_t stream_cap_words;
    void *index_dev;          /* 8-byte aligned */
    uint64_t index_cap_bytes;
} entro_encode_job;

entro_status entro_quantize_histogram_batched(const entro_quantize_job *jobs_host, int njobs,
                                              entro_qparams *qp_host, uint64_t *counts_host,
                                              void *cuda_stream);
entro_status entro_encode_batched(const entro_encode_job *jobs_host, int njobs, uint64_t *total_bits_host,
                                  void *cuda_stream);

/*
 * Parallel decode fused with dequantisation (Section 3, "Segmentation for parallel
 * Huffman decoding": every segment decodes independently from its known boundary; Eq. 1
 * inverted): out[i] = fp16_rne( s *_fp32 (float)(q[i] - z) ), q the decoded symbols in
 * element order.  Asynchronous on cuda_stream.  Malformed input (index not matching the
 * stream, a bit pattern that is no codeword) never faults: the affected chunk's output is
 * unspecified but in bounds, and the error is reported by entro_last_device_status.
 * n = 0: ENTRO_OK, nothing written.
 */
entro_status entro_decode_dequant(const uint32_t *stream_dev, uint64_t stream_words,
                                  const void *index_dev, uint64_t n, uint32_t chunk_symbols,
                                  const entro_codebook *cb_host, float scale, int32_t zero_point,
                                  void *out_fp16_dev, void *cuda_stream);

/*
 * The same for a whole model in one pass: all tensors' chunks form one work list that a
 * persistent kernel consumes (the paper balances load by dealing many segments to each
 * thread, Section 3).  descs_host is read before the call returns.  Asynchronous.
 * A call is: upload of the descriptors, construction of the per-tensor decode tables, the
 * decode launch.  For calls of at most ENTRO_STATIC_MAX_TENSORS descriptors the library
 * remembers the call: if the next call that uses its device area is the same call again
 * (byte-identical descriptors, same launch shape), descriptors and tables are found in
 * place and the call is the decode launch alone (a tensor decoded again and again, e.g. a
 * layer materialised on demand).
 */
entro_status entro_decode_dequant_batched(const entro_tensor_desc *descs_host, int ntensors,
                                          void *cuda_stream);

/*
 * Parallel decode to integers, the form in which the paper's decoder hands the weights to
 * its inference engine (Section 4: the engine works on the packed low-bit values).  Same
 * descriptors as entro_decode_dequant_batched; scale and zero_point are not used, and
 * out_fp16_dev points to bytes instead of fp16 values (16-byte aligned):
 *   packed = 0: n bytes, one symbol per byte;
 *   packed = 1: ceil(n / 2) bytes, symbol 2i in the low nibble of byte i and symbol 2i + 1
 *               in the high one (alphabets of at most 16 symbols; chunk_symbols even).
 * Asynchronous; errors as for the decode calls.
 */
entro_status entro_decode_symbols_batched(const entro_tensor_desc *descs_host, int ntensors, int packed,
                                          void *cuda_stream);

/* Host-resident input and output for one tensor of entro_decode_dequant_batched_host. */
typedef struct {
    const uint32_t *stream_host;  /* stream_words words (pinned memory for full speed) */
    const void *index_host;       /* entro_index_bytes bytes */
    void *out_fp16_host;          /* n fp16 values, or NULL: the result stays in out_fp16_dev only */
} entro_host_io;

/*
 * End-to-end form with host buffers: for every tensor, copy stream and index from
 * io_host[i] to the device buffers named in descs_host[i], decode + dequantise, and copy
 * the fp16 result back to io_host[i].out_fp16_host (where that is NULL the result is left
 * on the device: loading a compressed model from host memory).  The work is ordered after what
 * cuda_stream already holds; inside the call, uploads, decodes and downloads of different
 * groups of tensors overlap on two copy streams of the library's own.  Returns after
 * everything has completed (synchronises cuda_stream).
 */
entro_status entro_decode_dequant_batched_host(const entro_tensor_desc *descs_host,
                                               const entro_host_io *io_host, int ntensors,
                                               void *cuda_stream);

/* The matrix-vector side of one tensor of entro_decode_dequant_gemv.  Host struct; the
 * pointers inside are device pointers. */
typedef struct {
    uint32_t rows, cols;        /* W is [rows, cols] row-major, rows * cols = the tensor's n */
    const void *x_fp16_dev;     /* [batch][cols] fp16 values, token after token, 16-byte aligned */
    void *y_fp16_dev;           /* [batch][rows] fp16 results */
    uint32_t batch;             /* tokens, 1 .. ENTRO_GEMV_MAX_BATCH */
    uint32_t reserved;          /* 0 */
} entro_gemv_io;

/*
 * Decode + dequantise + matrix-vector product in one pass, for one token or a small batch,
 * without ever writing the fp16 weights: y[b][o] = fp16_rne( sum_i w_hat[o, i] * x[b][i] ),
 * w_hat = fp16(s * (q - z)) as in entro_decode_dequant, products and sums in fp32.  This is
 * the token-generation use of compressed weights: the paper puts its generation speed-up
 * down to the smaller amount of weight data that is moved while tokens are generated, a
 * phase bound by memory bandwidth (Section 4, Table 3); here only the compressed stream
 * crosses HBM, once for all tokens of the batch.  descs_host[i].out_fp16_dev is not used and may be NULL.  All ntensors
 * products are independent and run in one launch, which also rounds and stores y: a row that
 * lies inside one chunk is summed by one warp in a fixed order; a row that spans chunks gets
 * the chunks' partial sums added with fp32 atomics (the last chunk to arrive rounds), so its
 * result can differ from run to run in the last bits before the final rounding.
 * Limits: cols a multiple of 256, batch * cols at most 32768 (x of all tokens is staged in
 * shared memory), chunk_symbols a multiple of 256 (ENTRO_ERR_UNSUPPORTED otherwise); batch
 * outside 1 .. ENTRO_GEMV_MAX_BATCH or reserved != 0 is ENTRO_ERR_INVALID_ARG.
 * Asynchronous; malformed input is reported through entro_last_device_status as for the
 * decode calls.
 */
entro_status entro_decode_dequant_gemv(const entro_tensor_desc *descs_host, const entro_gemv_io *io_host,
                                       int ntensors, void *cuda_stream);

/*
 * The same products prepared once and run many times: the token-generation loop decodes the
 * same compressed weights for every token (Section 4, Table 3, token-generation rows), so
 * everything that does not change from token to token is set up once.  entro_gemv_prepare
 * validates the arguments as entro_decode_dequant_gemv does, allocates a device area of its
 * own for the plan (descriptors, decode tables, fp32 sums of the rows that span chunks),
 * fills it, and returns after cuda_stream has finished that work.  The compressed streams, x and y are NOT copied: the plan keeps the
 * device pointers given in descs_host / io_host, and every run reads the streams and x and
 * writes y there (the application refreshes x between runs).
 * entro_gemv_run is one kernel launch on cuda_stream (asynchronous): decode, multiply, round
 * and store y.  Runs of one plan must not overlap on the GPU (order them on one stream or
 * with events); different plans may.  Malformed input is reported through
 * entro_last_device_status; after such a report the plan's sums are undefined: release it
 * and prepare again.
 * entro_gemv_release waits for the device to finish with the plan's area and frees it
 * (NULL is allowed).
 */
typedef struct entro_gemv_plan entro_gemv_plan;
entro_status entro_gemv_prepare(const entro_tensor_desc *descs_host, const entro_gemv_io *io_host,
                                int ntensors, void *cuda_stream, entro_gemv_plan **plan_out);
entro_status entro_gemv_run(entro_gemv_plan *plan, void *cuda_stream);
entro_status entro_gemv_release(entro_gemv_plan *plan);

/*
 * Plain fp16 matrix-vector product y = fp16_rne(W x), W [rows, cols] row-major fp16 on the
 * device, fp32 products and sums: the step that follows an unfused decode, provided so that
 * "decode, then multiply" can be timed against the fused call.  cols a multiple of 8; w and
 * x 16-byte aligned.  Asynchronous.
 */
entro_status entro_gemv_fp16(const void *w_fp16_dev, uint32_t rows, uint32_t cols, const void *x_fp16_dev,
                             void *y_fp16_dev, void *cuda_stream);

/*
 * entro_decode_dequant_batched for callers that cannot allocate device memory.  (The paper
 * has no counterpart; this entry point exists for the sake of the host application.)
 *
 * The other decode calls keep their descriptors and decode tables in a workspace that the
 * library obtains with cudaMalloc / cudaMallocHost on first use and re-allocates when a
 * larger model arrives.  That is unusable where the application has already handed all
 * device memory to its own pool, where an allocation (which synchronises the whole device)
 * would stall kernels running on other streams, or where the CUDA allocator must not be
 * entered at all.  This variant calls no allocator: descriptors travel as kernel
 * arguments, and tables, work counter and status word live in an array that is part of the
 * library's device image (about 575 KB, held on every GPU that loads the library until
 * the process exits).
 *
 *  - At most ENTRO_STATIC_MAX_TENSORS tensors with n > 0 per call; more returns
 *    ENTRO_ERR_TOO_MANY_TENSORS and launches nothing.  Decode a larger model in slices.
 *  - The first call on each device looks up the array's device address (that device must
 *    be current, as for every call); make that first call outside any stream capture.
 *  - All calls on a device share the one array, and it keeps what the previous call left:
 *    each call rewrites what it uses and clears its counter and status first.  Two calls
 *    whose kernels overlap on the GPU (different streams, no event between them) race on
 *    it; keep them on one stream or order them.
 *  - status_dev: NULL, or a device pointer to one uint32_t that receives 0 if every chunk
 *    decoded cleanly and a non-zero value if stream, index and codebook disagreed
 *    (written asynchronously on cuda_stream; entro_last_device_status does not see this
 *    call).  Output, alignment rules and error behaviour are otherwise those of
 *    entro_decode_dequant_batched.  Asynchronous.
 */
entro_status entro_decode_dequant_static(const entro_tensor_desc *descs_host, int ntensors,
                                         uint32_t *status_dev, void *cuda_stream);

/*
 * Synchronise cuda_stream, then report and clear what decode kernels found since the last
 * call: ENTRO_OK or ENTRO_ERR_CORRUPT_STREAM (ENTRO_ERR_CUDA if the stream itself failed).
 */
entro_status entro_last_device_status(void *cuda_stream);

/*
 * Launch shape of the decode kernel; every argument may be 0 to keep its current value.
 *   lut_bits: window of the eight-symbol table used for alphabets of <= 16 symbols (10 .. 12)
 *   warps_per_cta: 4 .. 32;  ctas_per_sm: 1 .. 8;  chunks_per_item: largest number of 4096-symbol
 *   chunks a CTA claims at once (the library shrinks it for small launches, for the last
 *   part of a large one, and in proportion for larger chunks)
 * ENTRO_ERR_INVALID_ARG (nothing changed) if a value is out of range or the shape does
 * not fit in shared memory.
 */
entro_status entro_set_decode_config(int lut_bits, int warps_per_cta, int ctas_per_sm,
                                     int chunks_per_item);

/*
 * Optional timing of the decode kernel alone (CUDA events recorded on the caller's stream
 * right before and after its launch).  entro_profile_begin(max_records) arms up to
 * max_records recordings on the current device (0 disarms); every batched decode then
 * fills the next record.  entro_profile_read waits for the recorded launches, writes their
 * durations in milliseconds to ms_host (at most cap), re-arms, and returns how many it
 * wrote (-1 on error).
 */
entro_status entro_profile_begin(int max_records);
int entro_profile_read(float *ms_host, int cap);

/*
 * The checked build (compiled with -DENTRO_CHECKED: python -m paper_2505_02380_b200.build
 * --checked makes libentro_checked.so) tests, before each access, every address that the
 * decode kernel works out by hand: shared-memory offsets of table cells, ring words, index
 * slots and staged x; place and extent of every bulk copy; every output store.  A violation
 * is counted and the access left out; nothing traps and no wait is unbounded.  It stands
 * in for a memory checker and runs several times slower.  entro_checked_build: 1 in that
 * build, else 0.  entro_check_violations: waits for the device, then returns and clears the
 * count on the current device (always 0 in the ordinary build, -1 on a CUDA error).
 */
int entro_checked_build(void);
long long entro_check_violations(void);

/* Kernels launched by this library on the calling thread's device since load (for
 * launch accounting in benchmarks). */
uint64_t entro_kernel_launch_count(void);

const char *entro_status_string(entro_status st);

#ifdef __cplusplus
}
#endif
#endif /* ENTRO_H */
