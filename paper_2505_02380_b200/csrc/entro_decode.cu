// Parallel Huffman decode fused with dequantisation to fp16 (Section 3, "Segmentation for
// parallel Huffman decoding"; Eq. 1 inverted).
//
// Work split: a chunk (one segment) is decoded by one warp, each lane owning one of the
// chunk's 32 sub-blocks.  The lanes' start positions come from a warp prefix sum over the
// sub-block bit lengths stored in the index.  The warp stages the chunk's bytes into
// shared memory with one bulk asynchronous copy (the next chunk's bytes are prefetched
// into L2 meanwhile), every lane then walks its own bits with shared-memory lookup tables
// whose entries already hold dequantised fp16 values, and the results leave through a
// swizzled shared-memory tile as coalesced 16-byte-per-lane stores.  A persistent grid
// pulls work items (runs of chunks of one tensor) from a global counter; the warps of a
// CTA share out an item's chunks through a shared-memory counter.
//
// Tables per tensor (built by build_tables_kernel, cached in shared memory per CTA):
//   lut1  2^K entries indexed by the next K stream bits.
//         alphabets > 16 symbols: one symbol per entry,  value << 16 | length, or kEscFlag
//         alphabets <= 16 symbols: four symbols per entry, nibbles << 8 | total length, or
//         kQuadEscFlag; the fp16 values come from a 256-entry table of symbol pairs
//   lut2  second level for codes longer than K (single-symbol mode): indexed by
//         (window - t2) >> shift2, same entry format
//   aux   canonical ranges per length for whatever neither table resolves
#include <cuda_fp16.h>

#include "entro_internal.h"

namespace entro {
namespace {

constexpr int kTile = 32;                 // symbols per lane between two flushes of the output tile
constexpr int kTileBytes = 32 * kTile * 2;
constexpr int kUnits = kTile / 8;         // 16-byte units per tile row
constexpr uint32_t kWaitTries = 1u << 16; // bound on polling a bulk copy (each try may suspend)
constexpr uint32_t kLut2MaxBits = 20;     // longest code the second level resolves

// ------------------------------------------------------------------ table construction

__device__ __forceinline__ uint32_t range_decode(const DecodeAux& aux, uint32_t window, uint32_t max_l, uint32_t& len)
{
    // smallest l with window < limit[l]; the symbol is the (code - first_code)-th of that length
    for (uint32_t l = 1; l <= max_l; ++l) {
        if ((unsigned long long)window < aux.limit[l]) {
            len = l;
            return aux.sorted[(aux.offset[l] + ((window >> (32 - l)) - aux.first_code[l])) & 0xffu];
        }
    }
    len = 0;
    return 0;
}

// One block per tensor.
__global__ void __launch_bounds__(256) build_tables_kernel(const DevTensor* __restrict__ tensors, int lut_bits,
                                                           TensorTables* __restrict__ tables,
                                                           uint32_t* __restrict__ control)
{
    __shared__ DecodeAux aux;
    __shared__ uint32_t count[ENTRO_MAX_CODE_LEN + 1];
    __shared__ uint8_t len[ENTRO_MAX_SYMBOLS];
    const int t = blockIdx.x;
    const int tid = threadIdx.x;
    const DevTensor& T = tensors[t];
    TensorTables& out = tables[t];
    if (t == 0 && tid == 0) control[0] = 0;   // work counter of the decode kernel that follows
    if (tid <= ENTRO_MAX_CODE_LEN) count[tid] = 0;
    len[tid] = (uint32_t)tid < T.nsym ? T.len[tid] : 0;
    __syncthreads();
    const uint32_t l = len[tid];
    if (l) atomicAdd(&count[l], 1u);
    __syncthreads();
    if (tid == 0) {
        unsigned long long code = 0;   // reaches 2^32 after the last length of a complete code
        uint32_t off = 0, max_len = 0;
        aux.limit[0] = 0;
        aux.first_code[0] = 0;
        aux.offset[0] = 0;
        for (int k = 1; k <= ENTRO_MAX_CODE_LEN; ++k) {
            code <<= 1;
            aux.first_code[k] = (uint32_t)code;
            aux.offset[k] = off;
            code += count[k];
            off += count[k];
            aux.limit[k] = code << (32 - k);
            if (count[k]) max_len = k;
        }
        aux.max_len = max_len;
        aux.quad = T.nsym <= 16 ? 1u : 0u;
        // second level: windows at or above the end of the codes that fit the first level
        aux.t2 = 0;
        aux.shift2 = 0;
        aux.n2 = 0;
        const unsigned long long t2 = aux.limit[lut_bits];
        if (!aux.quad && max_len > (uint32_t)lut_bits && t2 < (1ull << 32)) {
            uint32_t bits = max_len < kLut2MaxBits ? max_len : kLut2MaxBits;
            for (; bits > (uint32_t)lut_bits; --bits) {
                unsigned long long n = ((1ull << 32) - t2 + (1ull << (32 - bits)) - 1) >> (32 - bits);
                if (n <= (unsigned long long)kLut2Entries) {
                    aux.t2 = (uint32_t)t2;
                    aux.shift2 = 32 - bits;
                    aux.n2 = (uint32_t)n;
                    break;
                }
            }
        }
        aux.pad[0] = aux.pad[1] = aux.pad[2] = 0;
    }
    __syncthreads();
    if (l) {
        uint32_t rank = 0;
        for (int k = 0; k < tid; ++k) rank += (len[k] == l);
        aux.sorted[aux.offset[l] + rank] = (uint8_t)tid;
    }
    const float d = (float)(tid - T.zero_point);
    aux.val[tid] = __half_as_ushort(__float2half_rn(__fmul_rn(T.scale, d)));
    __syncthreads();
    {
        uint32_t used = aux.offset[ENTRO_MAX_CODE_LEN] + count[ENTRO_MAX_CODE_LEN];
        if ((uint32_t)tid >= used) aux.sorted[tid] = 0;   // never indexed; keep it defined
    }
    __syncthreads();

    const uint32_t entries = 1u << lut_bits;
    if (aux.quad) {
        for (uint32_t i = tid; i < entries; i += 256) {
            uint32_t window = i << (32 - lut_bits);
            uint32_t used = 0, nibbles = 0;
            bool ok = true;
            for (int k = 0; k < 4; ++k) {
                uint32_t sl;
                uint32_t sym = range_decode(aux, window, (uint32_t)lut_bits - used, sl);
                if (sl == 0) {
                    ok = false;
                    break;
                }
                nibbles |= sym << (4 * k);
                used += sl;
                window <<= sl;   // sl <= lut_bits < 32
            }
            out.lut1[i] = ok ? ((nibbles << 8) | used) : kQuadEscFlag;
        }
        // fp16 values of a pair of symbols: low nibble first
        out.lut2[tid] = (uint32_t)aux.val[tid & 15] | ((uint32_t)aux.val[tid >> 4] << 16);
    } else {
        for (uint32_t i = tid; i < entries; i += 256) {
            uint32_t sl;
            uint32_t sym = range_decode(aux, i << (32 - lut_bits), (uint32_t)lut_bits, sl);
            out.lut1[i] = sl ? (((uint32_t)aux.val[sym] << 16) | sl) : kEscFlag;
        }
        for (uint32_t i = tid; i < aux.n2; i += 256) {
            uint32_t sl;
            uint32_t sym = range_decode(aux, aux.t2 + (i << aux.shift2), 32 - aux.shift2, sl);
            out.lut2[i] = sl ? (((uint32_t)aux.val[sym] << 16) | sl) : kEscFlag;
        }
    }
    const uint32_t* src = reinterpret_cast<const uint32_t*>(&aux);
    uint32_t* dst = reinterpret_cast<uint32_t*>(&out.aux);
    for (uint32_t i = tid; i < sizeof(DecodeAux) / 4; i += 256) dst[i] = src[i];
}

// ------------------------------------------------------------------ bit reader

// 64-bit window, left-justified: `nb` valid bits, the rest zero.  `next` is the index of
// the next 32-bit word to pull in.
struct Reader {
    uint32_t hi, lo;
    int nb;
    uint32_t next;
};

struct SmemSource {
    const uint32_t* words;
    uint32_t last;            // highest index that may be read
    __device__ __forceinline__ uint32_t get(uint32_t i) const { return words[min(i, last)]; }
};

struct GlobalSource {
    const uint32_t* words;
    uint64_t count;           // words readable from `words`
    __device__ __forceinline__ uint32_t get(uint32_t i) const { return i < count ? __ldg(words + i) : 0u; }
};

template <class Src>
__device__ __forceinline__ void reader_init(Reader& r, const Src& src, uint32_t word, uint32_t bit)
{
    uint32_t w0 = src.get(word), w1 = src.get(word + 1);
    r.hi = __funnelshift_l(w1, w0, bit);          // bit < 32
    r.lo = __funnelshift_l(0u, w1, bit);
    r.nb = 64 - (int)bit;
    r.next = word + 2;
}

// Top up to more than 32 valid bits.  With nb <= 32 the low word is empty.
template <class Src>
__device__ __forceinline__ void reader_refill(Reader& r, const Src& src)
{
    if (r.nb <= 32) {
        uint32_t w = src.get(r.next);
        r.next++;
        r.hi |= __funnelshift_rc(w, 0u, (uint32_t)r.nb);
        r.lo = __funnelshift_lc(0u, w, (uint32_t)(32 - r.nb));
        r.nb += 32;
    }
}

// Drop `n` bits, 0 <= n <= 32.
__device__ __forceinline__ void reader_skip(Reader& r, uint32_t n)
{
    if (n >= 32) {
        r.hi = r.lo;
        r.lo = 0;
    } else {
        r.hi = __funnelshift_l(r.lo, r.hi, n);
        r.lo <<= n;
    }
    r.nb -= (int)n;
}

struct Tables {
    const uint32_t* lut1;      // shared
    const uint32_t* lut2;      // shared
    const DecodeAux* aux;      // shared
    uint32_t* status;          // global
};

// One symbol from a full 32-bit window by the canonical ranges; a pattern that is no
// codeword is flagged and dropped as a single bit.  Entry format: value << 16 | length.
__device__ __noinline__ uint32_t decode_by_range(const DecodeAux* aux, uint32_t window, uint32_t* status)
{
    uint32_t len;
    uint32_t sym = range_decode(*aux, window, aux->max_len, len);
    if (len == 0) {
        atomicOr(status, kStatCorrupt);
        return 1u;
    }
    return ((uint32_t)aux->val[sym] << 16) | len;
}

// A symbol the first level could not resolve: second level, then the ranges.
__device__ __forceinline__ uint32_t decode_long(const Tables& tb, uint32_t window)
{
    const DecodeAux* aux = tb.aux;
    if (window >= aux->t2) {
        uint32_t i = (window - aux->t2) >> aux->shift2;
        if (i < aux->n2) {
            uint32_t e = tb.lut2[i];
            if (!(e & kEscFlag)) return e;
        }
    }
    return decode_by_range(aux, window, tb.status);
}

// One symbol, any tensor mode (used off the fast path).
template <int K>
__device__ __forceinline__ uint32_t decode_one(const Tables& tb, uint32_t window)
{
    if (tb.aux->quad) return decode_by_range(tb.aux, window, tb.status);
    uint32_t e = tb.lut1[window >> (32 - K)];
    if (e & kEscFlag) e = decode_long(tb, window);
    return e;
}

// Out-of-line repair of a pair of lookups in which at least one hit an escape entry.  On
// entry the window stands before the first unresolved symbol (escape entries have length
// 0): before symbol 0 if e0 is an escape, else before symbol 1.
struct PairFix {
    Reader r;
    uint32_t e0, e1;
};

template <int K>
__device__ __noinline__ PairFix redo_pair(const uint32_t* lut1, const uint32_t* lut2, const DecodeAux* aux,
                                         uint32_t* status, const uint32_t* words, uint32_t last, Reader r,
                                         uint32_t e0)
{
    Tables tb{lut1, lut2, aux, status};
    SmemSource src{words, last};
    PairFix f;
    if (e0 & kEscFlag) {
        reader_refill(r, src);
        e0 = decode_long(tb, r.hi);
        reader_skip(r, e0 & 0xffu);
    }
    reader_refill(r, src);
    uint32_t e1 = lut1[r.hi >> (32 - K)];
    if (e1 & kEscFlag) e1 = decode_long(tb, r.hi);
    reader_skip(r, e1 & 0xffu);
    f.r = r;
    f.e0 = e0;
    f.e1 = e1;
    return f;
}

// The same for a four-symbol entry: the four symbols one by one.  Returns the two pair
// bytes (symbols 0,1 and 2,3) in e0, e1.
__device__ __noinline__ PairFix redo_quad(const DecodeAux* aux, uint32_t* status, const uint32_t* words,
                                         uint32_t last, Reader r)
{
    SmemSource src{words, last};
    PairFix f;
    uint32_t nib = 0;
    for (int k = 0; k < 4; ++k) {
        reader_refill(r, src);
        uint32_t len;
        uint32_t sym = range_decode(*aux, r.hi, aux->max_len, len);
        if (len == 0) {
            atomicOr(status, kStatCorrupt);
            len = 1;
        }
        reader_skip(r, len);
        nib |= (sym & 15u) << (4 * k);
    }
    f.r = r;
    f.e0 = nib & 0xffu;
    f.e1 = nib >> 8;
    return f;
}

// ------------------------------------------------------------------ bulk copy + mbarrier

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }

__device__ __forceinline__ void mbar_init(uint32_t bar, uint32_t count)
{
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(bar), "r"(count) : "memory");
}

__device__ __forceinline__ void bulk_load(uint32_t dst, const void* src, uint32_t bytes, uint32_t bar)
{
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(bar), "r"(bytes) : "memory");
    asm volatile("cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(dst),
                 "l"(src), "r"(bytes), "r"(bar)
                 : "memory");
}

__device__ __forceinline__ void bulk_prefetch_l2(const void* src, uint32_t bytes)
{
    asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(src), "r"(bytes) : "memory");
}

// Bounded wait for phase `parity` of the barrier; false if the bound ran out.  Each try may
// suspend the thread for up to the hinted time, so waiting costs few issue slots.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    for (uint32_t tries = 0; tries < kWaitTries; ++tries) {
        uint32_t done;
        asm volatile(
            "{\n\t.reg .pred p;\n\t"
            "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
            "selp.u32 %0, 1, 0, p;\n\t}"
            : "=r"(done)
            : "r"(bar), "r"(parity), "r"(20000u)
            : "memory");
        if (done) return true;
    }
    return false;
}

// ------------------------------------------------------------------ one chunk

struct WarpCtx {
    Tables tb;
    uint32_t* stage;           // shared, this warp's compressed bytes
    uint4* tile;               // shared, this warp's output tile
    uint32_t bar;              // shared address of this warp's mbarrier
    uint32_t stage_bytes;
    uint32_t phase;
    bool dead;                 // a bulk copy never completed: stop using the stage buffer
};

// Byte range of the stream that decoding chunk c touches, or false if the index does not
// describe a range inside the stream buffer.  A lane may look 12 bytes past its end.
__device__ __forceinline__ bool chunk_range(const DevTensor& T, uint64_t off0, uint64_t off1, uint64_t& byte0,
                                            uint64_t& byte1)
{
    byte0 = (off0 >> 3) & ~15ull;
    byte1 = ((off1 >> 3) + 13 + 15) & ~15ull;
    return off1 >= off0 && off1 - off0 <= 32ull * 65535ull && byte1 <= T.stream_words * 4;
}

// General path: any symbol count per lane, words fetched straight from global memory,
// scalar stores.  Used for the ragged last chunk of a tensor and for chunks whose bytes do
// not fit the stage buffer.
template <int K>
__device__ __noinline__ void decode_chunk_general(Tables tb, const DevTensor& T, uint32_t c, uint64_t off0,
                                                  uint32_t excl, uint32_t my_bits, uint32_t lane)
{
    const uint32_t sub = T.chunk_symbols / kSubBlocks;
    const uint64_t chunk_first = (uint64_t)c * T.chunk_symbols;
    const uint64_t chunk_syms = min((uint64_t)T.chunk_symbols, T.n - chunk_first);
    const uint64_t lane_first = (uint64_t)lane * sub;
    const uint32_t cnt = lane_first >= chunk_syms ? 0u : (uint32_t)min((uint64_t)sub, chunk_syms - lane_first);
    const uint64_t pos = off0 + excl;
    const uint64_t word0 = pos >> 5;
    GlobalSource src{T.stream + word0, word0 < T.stream_words ? T.stream_words - word0 : 0ull};
    Reader r;
    reader_init(r, src, 0u, (uint32_t)(pos & 31));
    uint16_t* out = T.out + chunk_first + lane_first;
    for (uint32_t i = 0; i < cnt; ++i) {
        reader_refill(r, src);
        uint32_t e = decode_one<K>(tb, r.hi);
        reader_skip(r, e & 0xffu);
        out[i] = (uint16_t)(e >> 16);
    }
    const uint64_t used = ((uint64_t)r.next << 5) - (uint64_t)r.nb - (pos & 31);
    if (used != my_bits) atomicOr(tb.status, kStatCorrupt);
}

// Flush the warp's output tile: each instruction writes (32 / kUnits) rows of kTile * 2
// contiguous bytes; row r of the tile belongs to lane r's sub-block.
__device__ __forceinline__ void flush_tile(const uint4* tile, uint16_t* out_chunk, uint32_t sub, uint32_t t0,
                                           uint32_t lane)
{
#pragma unroll
    for (int i = 0; i < kUnits; ++i) {
        const uint32_t row = i * (32 / kUnits) + lane / kUnits;
        const uint32_t unit = lane % kUnits;
        const uint32_t swz = (row / (8 / kUnits)) % kUnits;
        uint4 v = tile[row * kUnits + (unit ^ swz)];
        uint4* dst = reinterpret_cast<uint4*>(out_chunk + (uint64_t)row * sub + t0) + unit;
        __stcs(dst, v);
    }
}

// Fast path: a full chunk whose bytes are staged in shared memory.
template <int K>
__device__ __forceinline__ void decode_chunk_staged(WarpCtx& cx, const DevTensor& T, uint32_t c, uint64_t off0,
                                                    uint64_t byte0, uint32_t copy_bytes, uint32_t excl,
                                                    uint32_t my_bits, uint32_t lane)
{
    const uint32_t sub = T.chunk_symbols / kSubBlocks;
    if (lane == 0)
        bulk_load(smem_addr(cx.stage), reinterpret_cast<const char*>(T.stream) + byte0, copy_bytes, cx.bar);
    bool ok = mbar_wait(cx.bar, cx.phase);
    ok = __all_sync(0xffffffffu, ok);
    if (!ok) {
        if (lane == 0) atomicOr(cx.tb.status, kStatTimeout);
        cx.dead = true;
        return;
    }
    cx.phase ^= 1u;

    const SmemSource src{cx.stage, copy_bytes / 4 - 1};
    const uint32_t pos = (uint32_t)(off0 - byte0 * 8) + excl;     // bit position inside the stage buffer
    Reader r;
    reader_init(r, src, pos >> 5, pos & 31);

    const uint32_t* lut1 = cx.tb.lut1;
    // tile row = lane, 16-byte units swizzled so that both the per-lane writes and the
    // row-wise reads of the flush touch every bank once
    const uint32_t row_swz = (lane / (8 / kUnits)) % kUnits;
    uint4* my_row = cx.tile + lane * kUnits;
    uint16_t* out_chunk = T.out + (uint64_t)c * T.chunk_symbols;

    if (cx.tb.aux->quad) {
        const uint32_t* pair_val = cx.tb.lut2;
        for (uint32_t t0 = 0; t0 < sub; t0 += kTile) {
#pragma unroll 1
            for (int g = 0; g < kUnits; ++g) {
                uint32_t packed[4];
#pragma unroll
                for (int h = 0; h < 2; ++h) {
                    reader_refill(r, src);
                    uint32_t e = lut1[r.hi >> (32 - K)];
                    r.hi = __funnelshift_l(r.lo, r.hi, e);
                    r.lo = __funnelshift_l(0u, r.lo, e);
                    r.nb -= (int)(e & 0xffu);
                    uint32_t b0 = __byte_perm(e, 0u, 0x4441);     // byte 1: symbols 0, 1
                    uint32_t b1 = __byte_perm(e, 0u, 0x4442);     // byte 2: symbols 2, 3
                    if (__builtin_expect(e & kQuadEscFlag, 0)) {
                        PairFix f = redo_quad(cx.tb.aux, cx.tb.status, src.words, src.last, r);
                        r = f.r;
                        b0 = f.e0;
                        b1 = f.e1;
                    }
                    packed[2 * h] = pair_val[b0];
                    packed[2 * h + 1] = pair_val[b1];
                }
                my_row[g ^ row_swz] = make_uint4(packed[0], packed[1], packed[2], packed[3]);
            }
            __syncwarp();
            flush_tile(cx.tile, out_chunk, sub, t0, lane);
            __syncwarp();
        }
    } else {
        for (uint32_t t0 = 0; t0 < sub; t0 += kTile) {
#pragma unroll 1
            for (int g = 0; g < kUnits; ++g) {
                uint32_t packed[4];
#pragma unroll
                for (int p = 0; p < 4; ++p) {
                    reader_refill(r, src);
                    uint32_t e0 = lut1[r.hi >> (32 - K)];
                    r.hi = __funnelshift_l(r.lo, r.hi, e0);
                    r.lo = __funnelshift_l(0u, r.lo, e0);
                    uint32_t e1 = lut1[r.hi >> (32 - K)];
                    r.hi = __funnelshift_l(r.lo, r.hi, e1);
                    r.lo = __funnelshift_l(0u, r.lo, e1);
                    r.nb -= (int)((e0 + e1) & 0xffu);
                    if (__builtin_expect((e0 | e1) & kEscFlag, 0)) {
                        PairFix f = redo_pair<K>(lut1, cx.tb.lut2, cx.tb.aux, cx.tb.status, src.words, src.last, r, e0);
                        r = f.r;
                        e0 = f.e0;
                        e1 = f.e1;
                    }
                    packed[p] = __byte_perm(e0, e1, 0x7632);      // two fp16 values, first symbol low
                }
                my_row[g ^ row_swz] = make_uint4(packed[0], packed[1], packed[2], packed[3]);
            }
            __syncwarp();
            flush_tile(cx.tile, out_chunk, sub, t0, lane);
            __syncwarp();
        }
    }
    const uint32_t used = (r.next << 5) - (uint32_t)r.nb - pos;
    if (used != my_bits) atomicOr(cx.tb.status, kStatCorrupt);
    __syncwarp();   // all lanes are done with the stage buffer before it is overwritten
}

// Decode chunk c; `next_c` (or 0xffffffff) is the chunk this warp will take afterwards, whose
// bytes are pulled into L2 while this one is being decoded.
template <int K>
__device__ __forceinline__ void decode_chunk(WarpCtx& cx, const DevTensor& T, uint32_t c, uint32_t next_c,
                                             uint32_t lane)
{
    const uint64_t off0 = T.offsets[c];
    const uint64_t off1 = T.offsets[c + 1];
    const uint32_t my_bits = T.sub_len[(uint64_t)c * kSubBlocks + lane];
    if (next_c < T.n_chunks && lane == 0) {
        uint64_t b0, b1;
        if (chunk_range(T, T.offsets[next_c], T.offsets[next_c + 1], b0, b1))
            bulk_prefetch_l2(reinterpret_cast<const char*>(T.stream) + b0, (uint32_t)(b1 - b0));
    }
    uint32_t incl = my_bits;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t t = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= (uint32_t)d) incl += t;
    }
    const uint32_t total = __shfl_sync(0xffffffffu, incl, 31);
    const uint32_t excl = incl - my_bits;

    uint64_t byte0, byte1;
    if (!chunk_range(T, off0, off1, byte0, byte1) || off1 - off0 != total) {
        if (lane == 0) atomicOr(cx.tb.status, kStatCorrupt);
        return;
    }
    const uint32_t sub = T.chunk_symbols / kSubBlocks;
    const bool full = (uint64_t)(c + 1) * T.chunk_symbols <= T.n;
    const uint64_t copy_bytes = byte1 - byte0;
    if (full && (sub % kTile) == 0 && copy_bytes <= cx.stage_bytes && !cx.dead)
        decode_chunk_staged<K>(cx, T, c, off0, byte0, (uint32_t)copy_bytes, excl, my_bits, lane);
    else
        decode_chunk_general<K>(cx.tb, T, c, off0, excl, my_bits, lane);
}

// ------------------------------------------------------------------ persistent kernel

// item_start[t] = first work item of tensor t, item_start[ntensors] = number of items; an
// item is up to chunks_per_item consecutive chunks of one tensor.
template <int K>
__global__ void __launch_bounds__(1024, 1) decode_kernel(const DevTensor* __restrict__ tensors, int ntensors,
                                                         const uint32_t* __restrict__ item_start,
                                                         const TensorTables* __restrict__ tables,
                                                         uint32_t chunks_per_item, uint32_t stage_bytes,
                                                         uint32_t* __restrict__ control)
{
    extern __shared__ __align__(128) unsigned char smem[];
    // layout: [lut1][lut2][aux][tensor][per-warp tile][per-warp stage][mbarriers][item + claim slots]
    uint32_t* s_lut1 = reinterpret_cast<uint32_t*>(smem);
    uint32_t* s_lut2 = s_lut1 + (1u << K);
    DecodeAux* s_aux = reinterpret_cast<DecodeAux*>(s_lut2 + kLut2Entries);
    DevTensor* s_tensor = reinterpret_cast<DevTensor*>(s_aux + 1);
    unsigned char* p = reinterpret_cast<unsigned char*>(s_tensor + 1);
    p = reinterpret_cast<unsigned char*>((reinterpret_cast<uintptr_t>(p) + 127) & ~(uintptr_t)127);
    const uint32_t warps = blockDim.x >> 5;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    unsigned char* tiles = p;
    unsigned char* stages = tiles + (size_t)warps * kTileBytes;
    unsigned long long* bars = reinterpret_cast<unsigned long long*>(stages + (size_t)warps * stage_bytes);
    volatile uint32_t* s_item = reinterpret_cast<volatile uint32_t*>(bars + warps);   // [2]
    uint32_t* s_claim = const_cast<uint32_t*>(s_item) + 2;                            // [2]

    WarpCtx cx;
    cx.tb = Tables{s_lut1, s_lut2, s_aux, control + 1};
    cx.tile = reinterpret_cast<uint4*>(tiles + (size_t)warp * kTileBytes);
    cx.stage = reinterpret_cast<uint32_t*>(stages + (size_t)warp * stage_bytes);
    cx.bar = smem_addr(bars + warp);
    cx.stage_bytes = stage_bytes;
    cx.phase = 0;
    cx.dead = false;

    if (lane == 0) mbar_init(cx.bar, 1);
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");

    const uint32_t total_items = item_start[ntensors];
    if (threadIdx.x == 0) {
        s_item[0] = atomicAdd(control, 1u);
        s_claim[0] = 0;
    }
    __syncthreads();
    int cur = -1;
    uint32_t slot = 0;
    while (true) {
        const uint32_t item = s_item[slot];
        if (item >= total_items) break;
        // claim the next item early; it is read after the barrier that ends this one
        if (threadIdx.x == 0) {
            s_item[slot ^ 1u] = atomicAdd(control, 1u);
            s_claim[slot ^ 1u] = 0;
        }
        // tensor of this item: last t with item_start[t] <= item
        int lo = 0, hi = ntensors - 1;
        while (lo < hi) {
            int mid = (lo + hi + 1) >> 1;
            if (__ldg(item_start + mid) <= item) lo = mid;
            else hi = mid - 1;
        }
        if (lo != cur) {
            cur = lo;
            const TensorTables* tt = tables + cur;
            const uint4* g1 = reinterpret_cast<const uint4*>(tt->lut1);
            uint4* s1 = reinterpret_cast<uint4*>(s_lut1);
            for (uint32_t i = threadIdx.x; i < (1u << K) / 4; i += blockDim.x) s1[i] = __ldg(g1 + i);
            const uint4* g2 = reinterpret_cast<const uint4*>(tt->lut2);
            uint4* s2 = reinterpret_cast<uint4*>(s_lut2);
            for (uint32_t i = threadIdx.x; i < kLut2Entries / 4; i += blockDim.x) s2[i] = __ldg(g2 + i);
            const uint4* ga = reinterpret_cast<const uint4*>(&tt->aux);
            uint4* sa = reinterpret_cast<uint4*>(s_aux);
            for (uint32_t i = threadIdx.x; i < sizeof(DecodeAux) / 16; i += blockDim.x) sa[i] = __ldg(ga + i);
            const uint4* gt = reinterpret_cast<const uint4*>(tensors + cur);
            uint4* st = reinterpret_cast<uint4*>(s_tensor);
            for (uint32_t i = threadIdx.x; i < sizeof(DevTensor) / 16; i += blockDim.x) st[i] = __ldg(gt + i);
            __syncthreads();
        }
        const DevTensor& T = *s_tensor;
        const uint32_t first = (item - __ldg(item_start + cur)) * chunks_per_item;
        const uint32_t count = min(chunks_per_item, T.n_chunks - first);
        // the warps share out the item's chunks; each keeps one claim ahead for the L2 prefetch
        uint32_t k = 0;
        if (lane == 0) k = atomicAdd(&s_claim[slot], 1u);
        k = __shfl_sync(0xffffffffu, k, 0);
        while (k < count) {
            uint32_t kn = 0;
            if (lane == 0) kn = atomicAdd(&s_claim[slot], 1u);
            kn = __shfl_sync(0xffffffffu, kn, 0);
            decode_chunk<K>(cx, T, first + k, kn < count ? first + kn : 0xffffffffu, lane);
            k = kn;
        }
        __syncthreads();   // tables may be replaced; s_item / s_claim [slot ^ 1] are now visible
        slot ^= 1u;
    }
    // A warp that gave up on a bulk copy lets it land (bounded) before its buffer goes away.
    if (cx.dead) (void)mbar_wait(cx.bar, cx.phase);
}

struct Shape {
    size_t smem;
    uint32_t stage_bytes;
};

// Shared memory of one CTA for a launch shape; stage_bytes == 0 if it cannot fit.
Shape shape_for(const DecodeConfig& cfg, int max_smem, uint32_t want_stage)
{
    size_t fixed = (4u << cfg.lut_bits) + 4u * kLut2Entries + sizeof(DecodeAux) + sizeof(DevTensor) + 128;
    size_t per_warp_fixed = kTileBytes + 8;
    size_t tail = 16;
    size_t budget = (size_t)max_smem / cfg.ctas_per_sm;
    if (cfg.ctas_per_sm > 1) budget -= 1024;   // per-CTA reservation of the driver
    Shape s{0, 0};
    if (budget < fixed + tail + cfg.warps_per_cta * (per_warp_fixed + 512)) return s;
    size_t avail = (budget - fixed - tail) / cfg.warps_per_cta - per_warp_fixed;
    uint32_t stage = (uint32_t)(avail & ~(size_t)127);
    if (stage > want_stage) stage = want_stage;
    s.stage_bytes = stage;
    s.smem = fixed + tail + cfg.warps_per_cta * (per_warp_fixed + stage);
    return s;
}

template <int K>
entro_status launch_decode(Workspace* ws, const DecodeConfig& cfg, const DevTensor* tensors, int ntensors,
                           const uint32_t* item_start, uint32_t total_items, const TensorTables* tables,
                           uint32_t want_stage, cudaStream_t s)
{
    Shape sh = shape_for(cfg, ws->max_smem_optin, want_stage);
    if (sh.stage_bytes == 0) return ENTRO_ERR_UNSUPPORTED;
    static int configured_smem[64] = {0};
    if ((int)sh.smem > configured_smem[ws->device]) {
        ENTRO_CUDA(cudaFuncSetAttribute(decode_kernel<K>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)sh.smem));
        configured_smem[ws->device] = (int)sh.smem;
    }
    uint32_t grid = (uint32_t)ws->sm_count * cfg.ctas_per_sm;
    if (grid > total_items) grid = total_items;
    const bool timed = ws->prof_used < ws->prof_cap;
    if (timed) ENTRO_CUDA(cudaEventRecord(ws->prof_start[ws->prof_used], s));
    decode_kernel<K><<<grid, cfg.warps_per_cta * 32, sh.smem, s>>>(tensors, ntensors, item_start, tables,
                                                                   (uint32_t)cfg.chunks_per_item, sh.stage_bytes,
                                                                   ws->control);
    count_launch();
    ENTRO_CUDA(cudaGetLastError());
    if (timed) ENTRO_CUDA(cudaEventRecord(ws->prof_stop[ws->prof_used++], s));
    return ENTRO_OK;
}

entro_status validate_desc(const entro_tensor_desc& d)
{
    if (d.n == 0) return ENTRO_OK;
    if (!d.stream_dev || !d.index_dev || !d.out_fp16_dev) return ENTRO_ERR_INVALID_ARG;
    if (!aligned(d.stream_dev, 16) || !aligned(d.index_dev, 8) || !aligned(d.out_fp16_dev, 16))
        return ENTRO_ERR_INVALID_ARG;
    if (d.chunk_symbols < kSubBlocks || d.chunk_symbols % kSubBlocks || d.chunk_symbols > ENTRO_MAX_CHUNK_SYMBOLS)
        return ENTRO_ERR_INVALID_ARG;
    if (!codebook_lengths_valid(&d.cb)) return ENTRO_ERR_INVALID_ARG;
    if (num_chunks(d.n, d.chunk_symbols) > 0x7fffffffull) return ENTRO_ERR_UNSUPPORTED;
    if (d.stream_words < ENTRO_STREAM_SLACK_WORDS + 1) return ENTRO_ERR_INVALID_ARG;
    return ENTRO_OK;
}

}  // namespace

// Upload descriptors, build the tables and run the persistent decode kernel.
entro_status decode_batched_locked(Workspace* ws, const entro_tensor_desc* descs, int ntensors, cudaStream_t s)
{
    const DecodeConfig cfg = decode_config();
    int live = 0;
    for (int i = 0; i < ntensors; ++i) {
        entro_status st = validate_desc(descs[i]);
        if (st != ENTRO_OK) return st;
        if (descs[i].n) live++;
    }
    if (live == 0) return ENTRO_OK;

    const size_t tensors_bytes = (size_t)live * sizeof(DevTensor);
    const size_t items_bytes = (((size_t)live + 1) * 4 + 15) & ~(size_t)15;
    const size_t upload_bytes = tensors_bytes + items_bytes;
    const size_t tables_bytes = (size_t)live * sizeof(TensorTables);
    if (!reserve_pinned(ws, upload_bytes)) return ENTRO_ERR_CUDA;
    if (!reserve_device(ws, upload_bytes + tables_bytes)) return ENTRO_ERR_CUDA;

    DevTensor* ht = static_cast<DevTensor*>(ws->pinned);
    uint32_t* hitems = reinterpret_cast<uint32_t*>(static_cast<char*>(ws->pinned) + tensors_bytes);
    uint64_t items = 0;
    uint32_t want_stage = 0;
    int k = 0;
    for (int i = 0; i < ntensors; ++i) {
        const entro_tensor_desc& d = descs[i];
        if (!d.n) continue;
        DevTensor& t = ht[k];
        const uint64_t nc = num_chunks(d.n, d.chunk_symbols);
        t.stream = d.stream_dev;
        t.offsets = static_cast<const uint64_t*>(d.index_dev);
        t.sub_len = reinterpret_cast<const uint16_t*>(t.offsets + nc + 1);
        t.out = static_cast<uint16_t*>(d.out_fp16_dev);
        t.stream_words = d.stream_words;
        t.n = d.n;
        t.chunk_symbols = d.chunk_symbols;
        t.n_chunks = (uint32_t)nc;
        t.nsym = (uint32_t)d.cb.nsym;
        t.scale = d.scale;
        t.zero_point = d.zero_point;
        t.pad[0] = t.pad[1] = t.pad[2] = 0;
        for (int j = 0; j < ENTRO_MAX_SYMBOLS; ++j) t.len[j] = j < d.cb.nsym ? d.cb.len[j] : 0;
        hitems[k] = (uint32_t)items;
        items += (nc + cfg.chunks_per_item - 1) / cfg.chunks_per_item;
        if (items > 0x7fffffffull) return ENTRO_ERR_UNSUPPORTED;
        // stage buffer: room for a chunk at one byte per symbol (an 8-bit alphabet averages
        // less), or 3/8 of a byte for alphabets of 16 symbols and fewer; chunks that need
        // more take the general path
        uint32_t want = d.cb.nsym <= 16 ? (d.chunk_symbols * 3) / 8 : d.chunk_symbols;
        want = ((want + 127) & ~127u) + 128;
        if (want > want_stage) want_stage = want;
        ++k;
    }
    hitems[live] = (uint32_t)items;

    char* base = static_cast<char*>(ws->dev);
    DevTensor* dt = reinterpret_cast<DevTensor*>(base);
    uint32_t* ditems = reinterpret_cast<uint32_t*>(base + tensors_bytes);
    TensorTables* dtables = reinterpret_cast<TensorTables*>(base + upload_bytes);
    ENTRO_CUDA(cudaMemcpyAsync(dt, ht, upload_bytes, cudaMemcpyHostToDevice, s));
    mark_pinned_in_use(ws, s);
    build_tables_kernel<<<live, 256, 0, s>>>(dt, cfg.lut_bits, dtables, ws->control);
    count_launch();
    ENTRO_CUDA(cudaGetLastError());
    switch (cfg.lut_bits) {
        case 10: return launch_decode<10>(ws, cfg, dt, live, ditems, (uint32_t)items, dtables, want_stage, s);
        case 11: return launch_decode<11>(ws, cfg, dt, live, ditems, (uint32_t)items, dtables, want_stage, s);
        case 12: return launch_decode<12>(ws, cfg, dt, live, ditems, (uint32_t)items, dtables, want_stage, s);
    }
    return ENTRO_ERR_UNSUPPORTED;
}

}  // namespace entro

using namespace entro;

extern "C" entro_status entro_decode_dequant_batched(const entro_tensor_desc* descs_host, int ntensors,
                                                     void* cuda_stream)
{
    if (ntensors < 0 || (ntensors > 0 && !descs_host)) return ENTRO_ERR_INVALID_ARG;
    if (ntensors == 0) return ENTRO_OK;
    for (int i = 0; i < ntensors; ++i) {
        entro_status st = validate_desc(descs_host[i]);
        if (st != ENTRO_OK) return st;
    }
    Guard g;
    Workspace* ws = workspace();
    if (!ws) return ENTRO_ERR_CUDA;
    return decode_batched_locked(ws, descs_host, ntensors, (cudaStream_t)cuda_stream);
}

extern "C" entro_status entro_decode_dequant(const uint32_t* stream_dev, uint64_t stream_words, const void* index_dev,
                                             uint64_t n, uint32_t chunk_symbols, const entro_codebook* cb, float scale,
                                             int32_t zero_point, void* out_fp16_dev, void* cuda_stream)
{
    if (!cb) return ENTRO_ERR_INVALID_ARG;
    entro_tensor_desc d;
    d.stream_dev = stream_dev;
    d.stream_words = stream_words;
    d.index_dev = index_dev;
    d.n = n;
    d.chunk_symbols = chunk_symbols;
    d.scale = scale;
    d.zero_point = zero_point;
    d.cb = *cb;
    d.out_fp16_dev = out_fp16_dev;
    return entro_decode_dequant_batched(&d, 1, cuda_stream);
}

extern "C" entro_status entro_decode_dequant_batched_host(const entro_tensor_desc* descs, const entro_host_io* io,
                                                          int ntensors, void* cuda_stream)
{
    if (ntensors < 0 || (ntensors > 0 && (!descs || !io))) return ENTRO_ERR_INVALID_ARG;
    if (ntensors == 0) return ENTRO_OK;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    for (int i = 0; i < ntensors; ++i) {
        if (!descs[i].n) continue;
        if (!io[i].stream_host || !io[i].index_host || !io[i].out_fp16_host) return ENTRO_ERR_INVALID_ARG;
        entro_status st = validate_desc(descs[i]);
        if (st != ENTRO_OK) return st;
    }
    for (int i = 0; i < ntensors; ++i) {
        const entro_tensor_desc& d = descs[i];
        if (!d.n) continue;
        ENTRO_CUDA(cudaMemcpyAsync(const_cast<uint32_t*>(d.stream_dev), io[i].stream_host, d.stream_words * 4,
                                   cudaMemcpyHostToDevice, s));
        ENTRO_CUDA(cudaMemcpyAsync(const_cast<void*>(d.index_dev), io[i].index_host,
                                   entro_index_bytes(d.n, d.chunk_symbols), cudaMemcpyHostToDevice, s));
    }
    {
        Guard g;
        Workspace* ws = workspace();
        if (!ws) return ENTRO_ERR_CUDA;
        entro_status st = decode_batched_locked(ws, descs, ntensors, s);
        if (st != ENTRO_OK) return st;
    }
    for (int i = 0; i < ntensors; ++i) {
        const entro_tensor_desc& d = descs[i];
        if (!d.n) continue;
        ENTRO_CUDA(cudaMemcpyAsync(io[i].out_fp16_host, d.out_fp16_dev, d.n * 2, cudaMemcpyDeviceToHost, s));
    }
    ENTRO_CUDA(cudaStreamSynchronize(s));
    return ENTRO_OK;
}

// ------------------------------------------------------------------ decode without allocation

namespace entro {
namespace {

// Everything the decode of up to ENTRO_STATIC_MAX_TENSORS tensors needs besides the
// caller's buffers.  One instance per device that loads the library, held until exit.
struct StaticScratch {
    DevTensor tensors[ENTRO_STATIC_MAX_TENSORS];
    uint32_t item_start[16];          // ENTRO_STATIC_MAX_TENSORS + 1 in use
    uint32_t control[16];             // [0] work counter, [1] status
    TensorTables tables[ENTRO_STATIC_MAX_TENSORS];
};
static_assert(ENTRO_STATIC_MAX_TENSORS + 1 <= 16, "item_start holds one entry per tensor plus the total");

static __device__ __align__(256) unsigned char g_static_scratch[sizeof(StaticScratch)];

// In host code g_static_scratch is only a handle for the runtime; the device address is
// looked up once per device and kept here.
struct StaticDevice {
    StaticScratch* scratch = nullptr;
    int sm_count = 0;
    int max_smem_optin = 0;
    bool ready = false;
};
StaticDevice g_static_device[64];

struct StaticUpload {
    DevTensor tensors[ENTRO_STATIC_MAX_TENSORS];
    uint32_t item_start[16];
    int live;
};

// Copies the descriptors from the kernel's parameter space into the scratch and clears the
// words that must start at zero (the previous call's contents are still there).
__global__ void __launch_bounds__(256) static_upload_kernel(const __grid_constant__ StaticUpload up,
                                                            StaticScratch* __restrict__ sc)
{
    const uint32_t* src = reinterpret_cast<const uint32_t*>(up.tensors);
    uint32_t* dst = reinterpret_cast<uint32_t*>(sc->tensors);
    const uint32_t words = (uint32_t)up.live * (uint32_t)(sizeof(DevTensor) / 4);
    for (uint32_t i = threadIdx.x; i < words; i += blockDim.x) dst[i] = src[i];
    if (threadIdx.x < 16) {
        sc->item_start[threadIdx.x] = up.item_start[threadIdx.x];
        sc->control[threadIdx.x] = 0;
    }
}

entro_status static_device(StaticDevice** out)
{
    int dev = -1;
    ENTRO_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= 64) return ENTRO_ERR_UNSUPPORTED;
    StaticDevice* sd = &g_static_device[dev];
    if (!sd->ready) {
        void* p = nullptr;
        ENTRO_CUDA(cudaGetSymbolAddress(&p, g_static_scratch));
        ENTRO_CUDA(cudaDeviceGetAttribute(&sd->sm_count, cudaDevAttrMultiProcessorCount, dev));
        ENTRO_CUDA(cudaDeviceGetAttribute(&sd->max_smem_optin, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev));
        sd->scratch = static_cast<StaticScratch*>(p);
        sd->ready = true;
    }
    *out = sd;
    return ENTRO_OK;
}

}  // namespace
}  // namespace entro

extern "C" entro_status entro_decode_dequant_static(const entro_tensor_desc* descs_host, int ntensors,
                                                    uint32_t* status_dev, void* cuda_stream)
{
    if (ntensors < 0 || (ntensors > 0 && !descs_host)) return ENTRO_ERR_INVALID_ARG;
    if (status_dev && !aligned(status_dev, 4)) return ENTRO_ERR_INVALID_ARG;
    int live = 0;
    for (int i = 0; i < ntensors; ++i) {
        entro_status st = validate_desc(descs_host[i]);
        if (st != ENTRO_OK) return st;
        if (descs_host[i].n) live++;
    }
    if (live > ENTRO_STATIC_MAX_TENSORS) return ENTRO_ERR_TOO_MANY_TENSORS;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    Guard g;
    StaticDevice* sd = nullptr;
    entro_status st = static_device(&sd);
    if (st != ENTRO_OK) return st;
    if (live == 0) {
        if (status_dev) ENTRO_CUDA(cudaMemsetAsync(status_dev, 0, sizeof(uint32_t), s));
        return ENTRO_OK;
    }
    const DecodeConfig cfg = decode_config();

    StaticUpload up;
    uint64_t items = 0;
    uint32_t want_stage = 0;
    int k = 0;
    for (int i = 0; i < ntensors; ++i) {
        const entro_tensor_desc& d = descs_host[i];
        if (!d.n) continue;
        DevTensor& t = up.tensors[k];
        const uint64_t nc = num_chunks(d.n, d.chunk_symbols);
        t.stream = d.stream_dev;
        t.offsets = static_cast<const uint64_t*>(d.index_dev);
        t.sub_len = reinterpret_cast<const uint16_t*>(t.offsets + nc + 1);
        t.out = static_cast<uint16_t*>(d.out_fp16_dev);
        t.stream_words = d.stream_words;
        t.n = d.n;
        t.chunk_symbols = d.chunk_symbols;
        t.n_chunks = (uint32_t)nc;
        t.nsym = (uint32_t)d.cb.nsym;
        t.scale = d.scale;
        t.zero_point = d.zero_point;
        t.pad[0] = t.pad[1] = t.pad[2] = 0;
        for (int j = 0; j < ENTRO_MAX_SYMBOLS; ++j) t.len[j] = j < d.cb.nsym ? d.cb.len[j] : 0;
        up.item_start[k] = (uint32_t)items;
        items += (nc + cfg.chunks_per_item - 1) / cfg.chunks_per_item;
        if (items > 0x7fffffffull) return ENTRO_ERR_UNSUPPORTED;
        uint32_t want = d.cb.nsym <= 16 ? (d.chunk_symbols * 3) / 8 : d.chunk_symbols;
        want = ((want + 127) & ~127u) + 128;
        if (want > want_stage) want_stage = want;
        ++k;
    }
    for (int j = live; j < 16; ++j) up.item_start[j] = (uint32_t)items;
    up.live = live;

    StaticScratch* sc = sd->scratch;
    static_upload_kernel<<<1, 256, 0, s>>>(up, sc);
    count_launch();
    ENTRO_CUDA(cudaGetLastError());
    build_tables_kernel<<<live, 256, 0, s>>>(sc->tensors, cfg.lut_bits, sc->tables, sc->control);
    count_launch();
    ENTRO_CUDA(cudaGetLastError());
    // launch_decode reads only these fields of a workspace; no timing records are taken here
    Workspace ws;
    cudaGetDevice(&ws.device);
    ws.sm_count = sd->sm_count;
    ws.max_smem_optin = sd->max_smem_optin;
    ws.control = sc->control;
    switch (cfg.lut_bits) {
        case 10: st = launch_decode<10>(&ws, cfg, sc->tensors, live, sc->item_start, (uint32_t)items, sc->tables, want_stage, s); break;
        case 11: st = launch_decode<11>(&ws, cfg, sc->tensors, live, sc->item_start, (uint32_t)items, sc->tables, want_stage, s); break;
        case 12: st = launch_decode<12>(&ws, cfg, sc->tensors, live, sc->item_start, (uint32_t)items, sc->tables, want_stage, s); break;
        default: st = ENTRO_ERR_UNSUPPORTED;
    }
    if (st != ENTRO_OK) return st;
    if (status_dev)
        ENTRO_CUDA(cudaMemcpyAsync(status_dev, sc->control + 1, sizeof(uint32_t), cudaMemcpyDeviceToDevice, s));
    return ENTRO_OK;
}

extern "C" entro_status entro_set_decode_config(int lut_bits, int warps_per_cta, int ctas_per_sm, int chunks_per_item)
{
    Guard g;
    DecodeConfig c = decode_config();
    if (lut_bits) c.lut_bits = lut_bits;
    if (warps_per_cta) c.warps_per_cta = warps_per_cta;
    if (ctas_per_sm) c.ctas_per_sm = ctas_per_sm;
    if (chunks_per_item) c.chunks_per_item = chunks_per_item;
    if (c.lut_bits < 10 || c.lut_bits > kMaxLutBits || c.warps_per_cta < 4 || c.warps_per_cta > 32 ||
        c.ctas_per_sm < 1 || c.ctas_per_sm > 8 || c.chunks_per_item < 1 || c.chunks_per_item > 65536)
        return ENTRO_ERR_INVALID_ARG;
    Workspace* ws = workspace();
    if (ws) {
        // smallest useful stage buffer is 1 KiB
        Shape sh = shape_for(c, ws->max_smem_optin, 1024);
        if (sh.stage_bytes < 1024) return ENTRO_ERR_INVALID_ARG;
    }
    decode_config() = c;
    return ENTRO_OK;
}
