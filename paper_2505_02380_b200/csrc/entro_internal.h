// Internal declarations shared by the library's translation units (not installed).
#pragma once

#include <cuda_runtime.h>
#include <stdint.h>

#include "entro.h"

namespace entro {

constexpr int kSubBlocks = ENTRO_SUB_BLOCKS;
constexpr int kMaxLutBits = 12;               // widest window of the eight-symbol table
constexpr int kExpBitsMin = 4, kExpBitsMax = 9;   // mantissa bits of the exponent-indexed table, chosen per tensor
constexpr int kExpEntriesMax = 32 << kExpBitsMax; // 16384 cells of 4 bytes: the 64 KB the 32 copies of the smallest take
constexpr int kExpEntriesMin = 32 << kExpBitsMin;

// Device status bits (OR-ed by kernels, read by entro_last_device_status).
constexpr uint32_t kStatCorrupt = 1u;         // index / stream / codebook disagree
constexpr uint32_t kStatTimeout = 2u;         // a bounded wait on a bulk copy ran out
constexpr uint32_t kStatInternal = 4u;        // the kernel found its own assumptions about the device violated

// One tensor as the decode kernels see it.
struct DevTensor {
    const uint32_t* stream;
    const uint64_t* offsets;      // n_chunks + 1
    const uint16_t* sub_len;      // n_chunks * 32
    uint16_t* out;                // fp16 bit patterns
    uint64_t stream_words;
    uint64_t last_bit;            // a chunk may end at this stream bit at most: 28 bytes behind it are still inside the buffer
    uint64_t n;
    uint32_t chunk_symbols;
    uint32_t n_chunks;
    uint32_t nsym;
    float scale;
    int32_t zero_point;
    uint32_t item_chunks;         // chunks per work item of this tensor
    uint32_t raw_symbols;         // 1: the tables hold the symbols themselves, not dequantised values
    uint32_t full_chunks;         // chunks that hold chunk_symbols symbols (all but a ragged last one)
    uint32_t pad[2];
    uint8_t len[ENTRO_MAX_SYMBOLS];
};
static_assert(sizeof(DevTensor) % 16 == 0, "DevTensor is copied as 16-byte vectors");

// The matrix-vector side of one tensor for the fused decode + GEMV kernel.
struct GemvTensor {
    const uint16_t* x;    // [batch][cols] fp16 values
    float* y32;           // [batch][rows] fp32 accumulators of the rows that span chunks (workspace); zero between calls
    uint16_t* y;          // [batch][rows] fp16 results
    uint32_t rows, cols;
    uint32_t batch;       // tokens, 1 .. ENTRO_GEMV_MAX_BATCH
    uint32_t pad;
    uint32_t* pending;    // [rows] chunks that hold part of the row: expected << 16 | still to come
};
static_assert(sizeof(GemvTensor) == 48, "GemvTensor is read as three 16-byte vectors");
constexpr uint32_t kGemvMaxX = 32768;         // fp16 values of x (all tokens) staged in shared memory

// Per-tensor canonical-code description beside the lookup tables.
struct DecodeAux {
    unsigned long long limit[ENTRO_MAX_CODE_LEN + 1];  // left-justified end of the codes of length <= l
    uint32_t first_code[ENTRO_MAX_CODE_LEN + 1];
    uint32_t offset[ENTRO_MAX_CODE_LEN + 1];           // rank of the first symbol of length l
    uint16_t val[ENTRO_MAX_SYMBOLS];                   // fp16( s * (q - z) ) per symbol
    uint8_t sorted[ENTRO_MAX_SYMBOLS];                 // symbols by (length, symbol)
    uint32_t max_len;
    uint32_t oct;      // 1: eight symbols per lookup (alphabets of <= 16 symbols)
    uint32_t group;    // one-symbol lookups per group: 2, 3, 4; 8 = two groups of four under one check; 16 = eight on one view
    uint32_t expm;     // mantissa bits of this tensor's exponent-indexed table
    // worked out once per tensor so that a warp does not repeat it for every chunk:
    uint32_t key_mask;       // the bits of (float bits >> 12) that select a cell of the exponent-indexed table
    uint32_t key_lane_mask;  // lanes that share a copy of that table: copy = lane & this
    uint32_t turns;          // groups of 8 symbols per lane and full chunk (chunk_symbols / 256), 0 if chunks cannot be staged
    uint32_t mode;           // what the decode loop switches on: 0 = eight symbols per lookup, 9 / 17 = group 8 / 16 with an even number of turns per chunk, 18 = group 16 with turns in fours, else `group`
    unsigned long long index_src[20];   // lane l's 4 bytes of chunk 0's index entries: lanes 0..15 two sub-block lengths
                                        // each, lanes 16..19 the halves of offsets[c], offsets[c + 1]
};
static_assert(sizeof(DecodeAux) % 16 == 0, "DecodeAux is copied as 16-byte vectors");

// Everything the decode kernel loads into shared memory when it switches tensor.
struct TensorTables {
    // oct mode: eight fp16 values per window.  Otherwise the same 64 KB hold the exponent-indexed
    // table, 32 << aux.expm cells of value << 16 | length (length 64 = unresolved).
    uint4 oct_val[1u << kMaxLutBits];
    uint8_t oct_len[1u << kMaxLutBits];    // oct mode: bits the eight codes use, 0 = not eight whole codes
    uint32_t exp_small[kExpEntriesMin];    // oct mode: 4-bit-mantissa exponent-indexed table for the repair path
    DecodeAux aux;
    __host__ __device__ uint32_t* exp_lut() { return reinterpret_cast<uint32_t*>(oct_val); }
    __host__ __device__ const uint32_t* exp_lut() const { return reinterpret_cast<const uint32_t*>(oct_val); }
};
static_assert(sizeof(TensorTables) % 16 == 0, "TensorTables is copied as 16-byte vectors");
static_assert(sizeof(uint4) * (1u << kMaxLutBits) >= 4u * kExpEntriesMax, "the large exponent table shares the oct values' space");

struct DecodeConfig {
    int lut_bits = 12;
    int warps_per_cta = 32;
    int ctas_per_sm = 1;
    int chunks_per_item = 1792;
};

// Where the decode kernel sends the decoded values.
enum Sink : int {
    kSinkFp16 = 0,      // dequantised fp16 values to the output tensor
    kSinkGemv = 1,      // dequantised fp16 values into a matrix-vector product, one token
    kSinkBytes = 2,     // the symbols, one per byte
    kSinkNibbles = 3,   // the symbols, two per byte, the earlier one in the low nibble
    kSinkGemv2 = 4,     // ... into the products with up to 2, 4, 8 tokens
    kSinkGemv4 = 5,
    kSinkGemv8 = 6
};
// Accumulators per lane of a matrix-vector sink (0: not such a sink).
template <int kSink>
constexpr int kGemvBatchOf = kSink == kSinkGemv ? 1 : kSink == kSinkGemv2 ? 2 : kSink == kSinkGemv4 ? 4 : kSink == kSinkGemv8 ? 8 : 0;

// Per-device workspace owned by the library.
struct Workspace {
    int device = -1;
    int sm_count = 0;
    int max_smem_optin = 0;
    // device
    void* dev = nullptr;
    size_t dev_bytes = 0;
    uint32_t* control = nullptr;      // [0] work counter, [1] status, [2..] scratch flags
    // pinned host
    void* pinned = nullptr;
    size_t pinned_bytes = 0;
    cudaEvent_t upload_done = nullptr; // last async read of `pinned` by the device
    bool upload_pending = false;
    // copy streams and events of the host-buffer entry point (made on first use)
    static constexpr int kCopyGroups = 48;
    cudaStream_t copy_in = nullptr, copy_out = nullptr;
    cudaEvent_t ev_in[kCopyGroups] = {}, ev_dec[kCopyGroups] = {}, ev_edge = nullptr;
    // What the device area holds if the last call that filled it was a batched decode of few
    // tensors: the call's descriptors (host copy) and what its launch needs.  A repeat of that
    // call finds descriptors and tables already in place and is one launch.  reserve_device
    // (every call that fills the area goes through it) forgets it.
    static constexpr int kKeptTensors = ENTRO_STATIC_MAX_TENSORS;
    uint32_t big_items = 0;    // set around a launch: its first so many work items are the full-size ones (0: none to stripe)
    bool kept = false;
    int kept_ntensors = 0, kept_live = 0, kept_sink = 0;
    uint32_t kept_items = 0;
    DecodeConfig kept_cfg;
    entro_tensor_desc kept_descs[kKeptTensors];
    // optional timing of the decode kernel (entro_profile_begin / entro_profile_read)
    cudaEvent_t* prof_start = nullptr;
    cudaEvent_t* prof_stop = nullptr;
    int prof_cap = 0;
    int prof_used = 0;
};

// Returns the workspace of the current device (creating it), or nullptr on a CUDA error.
Workspace* workspace();
// Grow the device / pinned areas to at least these sizes (contents are not preserved).
bool reserve_device(Workspace* ws, size_t bytes);
bool reserve_pinned(Workspace* ws, size_t bytes);
// Wait until the device has finished reading the pinned area from an earlier call.
bool wait_pinned_free(Workspace* ws);
void mark_pinned_in_use(Workspace* ws, cudaStream_t s);
void lock();
void unlock();
void count_launch(int n = 1);
DecodeConfig& decode_config();

struct Guard {
    Guard() { lock(); }
    ~Guard() { unlock(); }
};

inline bool aligned(const void* p, size_t a) { return (reinterpret_cast<uintptr_t>(p) & (a - 1)) == 0; }
inline uint64_t num_chunks(uint64_t n, uint32_t c) { return (n + c - 1) / c; }
bool codebook_lengths_valid(const entro_codebook* cb);

}  // namespace entro

#define ENTRO_CUDA(call)                                   \
    do {                                                   \
        cudaError_t e__ = (call);                          \
        if (e__ != cudaSuccess) return ENTRO_ERR_CUDA;     \
    } while (0)
