// One chunk of the decode kernel: bulk copy into the warp's ring, index slots, lane start
// positions, the general path, and what happens to the decoded values (store, integer
// output, matrix-vector product).  Included by entro_decode.cu only.
#pragma once

#include "entro_decode_reader.cuh"

namespace entro {
namespace {

// ------------------------------------------------------------------ bulk copy + mbarrier

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

// One try at phase `parity` of the barrier; may suspend the thread for up to the hinted time.
__device__ __forceinline__ bool mbar_try(uint32_t bar, uint32_t parity)
{
    uint32_t done;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2, %3;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(done)
        : "r"(bar), "r"(parity), "r"(20000u)
        : "memory");
    return done != 0u;
}

// Bounded wait for phase `parity` of the barrier; false if the bound ran out.  The bytes have
// nearly always arrived long before they are asked for, so the first try stands by itself and
// the loop is off the usual path.
__device__ __forceinline__ bool mbar_wait(uint32_t bar, uint32_t parity)
{
    if (__builtin_expect(mbar_try(bar, parity), 1)) return true;
#pragma unroll 1
    for (uint32_t tries = 1; tries < kWaitTries; ++tries)
        if (mbar_try(bar, parity)) return true;
    return false;
}

// ------------------------------------------------------------------ one chunk

// Fixed places in shared memory: [tables][aux][tensor][rings ...].
template <int K>
__device__ __forceinline__ DecodeAux* aux_ptr() { return reinterpret_cast<DecodeAux*>(smem + lut_bytes(K)); }
template <int K>
__device__ __forceinline__ DevTensor* tensor_ptr()
{
    return reinterpret_cast<DevTensor*>(smem + lut_bytes(K) + sizeof(DecodeAux));
}

// The matrix-vector kernel keeps two more things behind the tensor: its GemvTensor and x.
template <int K>
constexpr uint32_t kGemvDesc = lut_bytes(K) + (uint32_t)sizeof(DecodeAux) + (uint32_t)sizeof(DevTensor);
template <int K>
constexpr uint32_t kGemvX = kGemvDesc<K> + (uint32_t)sizeof(GemvTensor);
template <int K>
__device__ __forceinline__ GemvTensor* gemv_ptr() { return reinterpret_cast<GemvTensor*>(smem + kGemvDesc<K>); }
// Offset of the first ring: behind the tensor, or behind x_bytes of staged x (a multiple of 128).
template <int K>
constexpr uint32_t rings_offset(bool gemv, uint32_t x_bytes)
{
    return ((gemv ? kGemvX<K> + x_bytes : kGemvDesc<K>) + 127u) & ~127u;
}

// What a warp carries from chunk to chunk (kept small: it lives in registers across the
// decode loop).
struct WarpCtx {
    uint32_t stage_addr;       // shared-window address of this warp's ring for compressed bytes
    uint32_t bar;              // shared-window address of this warp's two mbarriers
    uint32_t idx_addr;         // shared-window address of this warp's two index slots
    uint32_t state;            // bulk copies issued so far; bit 31: a copy never completed, stop staging
    __device__ __forceinline__ bool dead() const { return (state >> 31) != 0u; }
};

// An index slot holds one chunk's index entries, fetched asynchronously two chunks ahead:
// the 32 sub-block lengths (64 bytes), then offsets[c] and offsets[c + 1].
constexpr uint32_t kSlotBytes = 80;

enum : uint32_t { kStaged = 0, kGeneral = 1, kSkip = 2 };

// Chunk whose bytes have been asked for.  meta packs what the staging needs so that every field
// comes out by one or two operations: bits 0..1 kind, bit 2 copy issued, bits 4..15 the ring
// offset (a multiple of 16, in place), bits 16..17 the ticket modulo 4, bits 20..31 the byte
// count (a multiple of 16, at most 65520) shifted up by 16.  Everything else is re-read from the
// chunk's index slot when it is decoded.
struct Ready {
    uint32_t c;                // or kNone
    uint32_t meta;
    __device__ __forceinline__ uint32_t at() const { return meta & 0xfff0u; }
    __device__ __forceinline__ uint32_t bytes() const { return (meta >> 16) & 0xfff0u; }
    __device__ __forceinline__ uint32_t ticket() const { return (meta >> 16) & 3u; }
    __device__ __forceinline__ uint32_t kind() const { return meta & 3u; }
    __device__ __forceinline__ bool issued() const { return (meta & 4u) != 0u; }
};
__device__ __forceinline__ uint32_t ready_meta(uint32_t at, uint32_t bytes, uint32_t ticket, uint32_t kind)
{
    return at | kind | ((bytes | (ticket & 3u)) << 16);
}

__device__ __forceinline__ unsigned long long lds64(uint32_t addr)
{
    if (ENTRO_CHECK(smem_ok(addr, 8u))) return 0ull;
    unsigned long long v;
    asm volatile("ld.shared.b64 %0, [%1];" : "=l"(v) : "r"(addr));
    return v;
}

// Ask for chunk c's index entries to be copied into the slot at shared address `slot`
// (lanes 0..15 two sub-block lengths each, lanes 16 and 17 one offset each).  Nothing is
// held in registers while the copies are in flight.
__device__ __forceinline__ void fetch_index(const DecodeAux* aux, const DevTensor& T, uint32_t c, uint32_t slot, uint32_t lane)
{
    if (c != kNone && ENTRO_CHECK(c < T.n_chunks && smem_ok(slot, 16u) && smem_ok(slot + kSlotBytes - 16u, 16u))) c = kNone;
    if (c != kNone && lane < 20u) {
        // 4 bytes per lane: lanes 0..15 the sub-block lengths (64 bytes per chunk), lanes 16..19 the two offsets (8 per chunk)
        unsigned long long src;
        asm("mad.wide.u32 %0, %1, %2, %3;" : "=l"(src) : "r"(c), "r"(lane < 16u ? 64u : 8u), "l"(aux->index_src[lane]));
        asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(slot + lane * 4u), "l"(src) : "memory");
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}

__device__ __forceinline__ void issue_copy(const WarpCtx& cx, const DevTensor& T, Ready& r, uint64_t byte0, uint32_t lane,
                                           uint32_t stage_bytes)
{
    // the copy lands inside this warp's ring, comes from inside the stream buffer, and both ends are 16-byte aligned
    const bool bad = ENTRO_CHECK(r.at() + r.bytes() <= stage_bytes && smem_ok(cx.stage_addr + r.at(), 16u) &&
                                 r.bytes() >= 16u && smem_ok(cx.stage_addr + r.at() + r.bytes() - 16u, 16u) &&
                                 (byte0 & 15ull) == 0ull && byte0 + r.bytes() <= T.stream_words * 4ull);
    if (lane == 0 && !bad)
        bulk_load(cx.stage_addr + r.at(), reinterpret_cast<const char*>(T.stream) + byte0, r.bytes(),
                  cx.bar + 8u * (r.ticket() & 1u));
    r.meta |= 4u;
}

// Bytes of the stream that decoding a chunk touches: from the 16-byte boundary below its
// first bit to 13 bytes past its last (a window looks ahead), rounded up to 16.
__device__ __forceinline__ void chunk_bytes(uint64_t off0, uint64_t off1, uint64_t& byte0, uint64_t& byte1)
{
    byte0 = (off0 >> 3) & ~15ull;
    byte1 = ((off1 >> 3) + 13 + 15) & ~15ull;
}

// Chunk c's offsets have arrived in `slot`: check them, find a place in the ring next to
// `prev` (the chunk decoded before this one, still undecoded), and start the bulk copy if
// that place is free already.  All lanes compute the same values.
__device__ __forceinline__ Ready prepare(WarpCtx& cx, const DevTensor& T, uint32_t turns, uint32_t stage_bytes,
                                         uint32_t* status, uint32_t c, uint32_t slot, const Ready& prev, uint32_t lane)
{
    Ready r;
    r.c = c;
    r.meta = ready_meta(0, 0, 0, kSkip);
    asm volatile("cp.async.wait_all;" ::: "memory");
    __syncwarp();
    if (c == kNone) return r;
    const uint64_t off0 = lds64(slot + 64u), off1 = lds64(slot + 72u);
    // (off1 < off0 wraps to a huge difference; off1 <= last_bit keeps the copied bytes inside the buffer)
    if (off1 - off0 > 32ull * 65535ull || off1 > T.last_bit) {
        if (lane == 0) atomicOr(status, kStatCorrupt);
        return r;
    }
    // the bytes decoding touches (chunk_bytes), their count in 32-bit arithmetic: the chunk is short
    const uint64_t byte0 = (off0 >> 3) & ~15ull;
    const uint32_t bytes = (((uint32_t)(off1 >> 3) + 13u + 15u) & ~15u) - (uint32_t)byte0;
    // a full chunk of whole groups of 8 per lane whose bytes fit the ring is staged
    if (c >= T.full_chunks || turns == 0u || bytes > stage_bytes || cx.dead()) {
        r.meta = ready_meta(0, 0, 0, kGeneral);
        return r;
    }
    // ring placement: at the other end of the ring from the previous chunk's bytes (chunks
    // alternate between the start and the end, so two chunks that fit together never wait for
    // one another, whatever their sizes), else at the start once the previous chunk has been
    // decoded
    uint32_t at = 0;
    bool now = true;
    if (prev.c != kNone && prev.kind() == kStaged) {
        const uint32_t p_at = prev.at(), p_end = p_at + prev.bytes();
        const uint32_t top = stage_bytes - bytes;          // a multiple of 16, as both are
        if (bytes <= p_at) at = 0;
        else if (top >= p_end) at = top;
        else now = false;
    }
    r.meta = ready_meta(at, bytes, cx.state, kStaged);
    cx.state++;
    if (now) issue_copy(cx, T, r, byte0, lane, stage_bytes);
    else if (lane == 0)   // no room yet: at least bring the bytes into L2 while the previous chunk is decoded
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(reinterpret_cast<const char*>(T.stream) + byte0),
                     "r"(bytes)
                     : "memory");
    return r;
}

// A chunk has added its part of a row that spans chunks to the row's fp32 sums.  The chunk
// that brings the row's count of parts still to come to zero rounds the sums to fp16, and
// leaves sums and count as the next call wants to find them (zero, and the full count).
__device__ __forceinline__ void row_part_done(const GemvTensor* G, uint32_t row)
{
    __threadfence();                                   // this chunk's additions are visible before the count moves
    const uint32_t before = atomicSub(G->pending + row, 1u);
    if ((before & 0xffffu) != 1u) return;
    __threadfence();
    for (uint32_t b = 0; b < G->batch; ++b) {
        const uint64_t at = (uint64_t)b * G->rows + row;
        G->y[at] = __half_as_ushort(__float2half_rn(atomicExch(G->y32 + at, 0.f)));
    }
    G->pending[row] = (before >> 16) * 0x10001u;
}

// Any symbol count per lane, words fetched straight from global memory, one value at a
// time: the ragged last chunk of a tensor, odd chunk sizes, chunks larger than the ring.
// With G set (kB > 0 accumulators) the values are not stored but multiplied into the
// matrix-vector products of the batch's tokens.
template <int kB>
__device__ __forceinline__ void decode_chunk_general(const DecodeAux* aux, uint32_t* status, const DevTensor& T,
                                                     const GemvTensor* G, int sink, uint32_t c, uint32_t excl,
                                                     uint32_t my_bits, uint32_t lane)
{
    const uint64_t chunk_first = (uint64_t)c * T.chunk_symbols;
    const uint32_t m = (uint32_t)min((uint64_t)T.chunk_symbols, T.n - chunk_first);   // symbols in the chunk
    const uint64_t pos = T.offsets[c] + excl;
    const uint64_t word0 = pos >> 5;
    GlobalWin r;
    r.words = T.stream + word0;
    r.count = word0 < T.stream_words ? T.stream_words - word0 : 0ull;
    const uint32_t bit = (uint32_t)(pos & 31);
    const uint32_t w0 = r.get(0), w1 = r.get(1);
    r.hi = __funnelshift_l(w1, w0, bit);
    r.lo = w1 << bit;
    r.nb = 64 - (int)bit;
    r.next = 2;
    const bool oct = aux->oct != 0;
    uint16_t* out = T.out + chunk_first;
    // this lane's symbols: groups lane, lane + 32, ... of 8 consecutive symbols
    for (uint32_t g = lane; g * 8u < m; g += kSubBlocks) {
        const uint32_t end = min(g * 8u + 8u, m);
        float acc[kB > 0 ? kB : 1];
#pragma unroll
        for (int b = 0; b < (kB > 0 ? kB : 1); ++b) acc[b] = 0.f;
        uint32_t low = 0;                       // the even symbol of a nibble pair
        for (uint32_t i = g * 8u; i < end; ++i) {
            gwin_refill(r);
            uint32_t e = kEscLen;
            if (!oct) e = exp_lookup(lut_key(aux, lane), ~r.hi);
            if ((e & 0xffffu) > 32u) e = decode_by_range(aux, r.hi, status);
            const uint32_t n = e & 0xffffu;
            r.hi = __funnelshift_lc(r.lo, r.hi, n);
            r.lo = __funnelshift_lc(0u, r.lo, n);
            r.nb -= (int)n;
            if (kB > 0) {
                const uint32_t col = (uint32_t)((chunk_first + i) % G->cols);
                const float v = __half2float(__ushort_as_half((uint16_t)(e >> 16)));
#pragma unroll
                for (int b = 0; b < kB; ++b)
                    if ((uint32_t)b < G->batch)
                        acc[b] = fmaf(v, __half2float(__ushort_as_half(__ldg(G->x + (uint64_t)b * G->cols + col))), acc[b]);
            } else if (sink == kSinkBytes) {
                reinterpret_cast<uint8_t*>(T.out)[chunk_first + i] = (uint8_t)(e >> 16);
            } else if (sink == kSinkNibbles) {
                // pairs never straddle a group of 8 and chunks hold an even number of symbols
                if (i & 1u) reinterpret_cast<uint8_t*>(T.out)[(chunk_first + i) >> 1] = (uint8_t)(low | ((e >> 16) << 4));
                else if (i + 1u == m) reinterpret_cast<uint8_t*>(T.out)[(chunk_first + i) >> 1] = (uint8_t)(e >> 16);
                else low = (e >> 16) & 15u;
            } else if (!ENTRO_CHECK(chunk_first + i < T.n)) {
                out[i] = (uint16_t)(e >> 16);
            }
        }
        // a group of 8 lies inside one row (cols is a multiple of 8)
        if (kB > 0) {
            const uint32_t row = (uint32_t)((chunk_first + g * 8u) / G->cols);
#pragma unroll
            for (int b = 0; b < kB; ++b)
                if ((uint32_t)b < G->batch) atomicAdd(G->y32 + (uint64_t)b * G->rows + row, acc[b]);
        }
    }
    const uint64_t used = ((uint64_t)r.next << 5) - (uint64_t)r.nb - bit;
    if (used != my_bits) atomicOr(status, kStatCorrupt);
    if (kB > 0) {
        // every row the chunk touches has now got this chunk's part
        __threadfence();
        __syncwarp();
        const uint32_t row0 = (uint32_t)(chunk_first / G->cols), row1 = (uint32_t)((chunk_first + m - 1u) / G->cols);
        for (uint32_t row = row0 + lane; row <= row1; row += kSubBlocks) row_part_done(G, row);
    }
}

// ------------------------------------------------------------------ what happens to decoded values

__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    if (ENTRO_CHECK(smem_ok(addr, 16u))) return make_uint4(0u, 0u, 0u, 0u);
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

// Where a lane's groups go in the output: group after group `stride` bytes apart (the 32
// lanes' groups of one step are contiguous), from `base`.  The address is formed by one
// multiply-add on the FMA pipe (the integer pipe is the busy one), and the byte offset
// doubles as the loop counter of the lane's sub-block.
struct OutCursor {
    const void* base;
    uint32_t off, end;
#ifdef ENTRO_CHECKED
    const char *lo, *hi;      // the output buffer of the tensor
#endif
    __device__ __forceinline__ void start(void* lane_first, uint32_t steps, uint32_t stride)
    {
        base = lane_first;
        off = 0;
        end = steps * stride;
    }
    // Checked build: the tensor's output is [first, first + bytes); is a store of n bytes at p inside it?
    __device__ __forceinline__ void bounds(const void* first, uint64_t bytes)
    {
#ifdef ENTRO_CHECKED
        lo = static_cast<const char*>(first);
        hi = lo + bytes;
#endif
    }
    __device__ __forceinline__ bool outside(const void* p, uint32_t n) const
    {
#ifdef ENTRO_CHECKED
        const char* c = static_cast<const char*>(p);
        return ENTRO_CHECK(c >= lo && c + n <= hi && (reinterpret_cast<uintptr_t>(p) & (n - 1u)) == 0u);
#else
        return false;
#endif
    }
    __device__ __forceinline__ bool more() const { return off != end; }
    __device__ __forceinline__ void* next(uint32_t stride)
    {
        unsigned long long a;
        asm("mad.wide.u32 %0, %1, 1, %2;" : "=l"(a) : "r"(off), "l"(base));
        off += stride;
        return reinterpret_cast<void*>(a);
    }
};

// Plain decode: the 8 values of this lane's next group go to the output tensor.  A lane's
// consecutive groups are 32 groups apart, so one call per lane writes 512 contiguous bytes.
struct EmitStore {
    static constexpr bool kTwice = true;    // a group may be written, found wrong, and written again
    OutCursor out;
    __device__ __forceinline__ void back(uint32_t groups) { out.off -= groups * 16u * kSubBlocks; }
    __device__ __forceinline__ bool more() const { return out.more(); }
    __device__ __forceinline__ void operator()(uint4 v)
    {
        uint4* p = static_cast<uint4*>(out.next(16u * kSubBlocks));
        if (!out.outside(p, 16u)) __stcs(p, v);
    }
    __device__ __forceinline__ void finish() {}
};

// Integer output (the form the paper's decoder produces): the tables hold the symbols
// themselves in their 16-bit value fields; a group of 8 leaves as 8 bytes ...
struct EmitBytes {
    static constexpr bool kTwice = true;
    OutCursor out;
    __device__ __forceinline__ void back(uint32_t groups) { out.off -= groups * 8u * kSubBlocks; }
    __device__ __forceinline__ bool more() const { return out.more(); }
    __device__ __forceinline__ void operator()(uint4 v)
    {
        uint2* p = static_cast<uint2*>(out.next(8u * kSubBlocks));
        if (!out.outside(p, 8u)) __stcs(p, make_uint2(__byte_perm(v.x, v.y, 0x6420), __byte_perm(v.z, v.w, 0x6420)));
    }
};

// ... or, for 4-bit symbols, as 4 bytes of two nibbles each, the earlier symbol low.
struct EmitNibbles {
    static constexpr bool kTwice = false;
    OutCursor out;
    __device__ __forceinline__ bool more() const { return out.more(); }
    __device__ __forceinline__ void operator()(uint4 v)
    {
        const uint32_t a = __byte_perm(v.x, v.y, 0x6420), b = __byte_perm(v.z, v.w, 0x6420);   // s0..s3, s4..s7
        const uint32_t ta = a | (a >> 4), tb = b | (b >> 4);                                   // bytes 0 and 2 hold the pairs
        uint32_t* p = static_cast<uint32_t*>(out.next(4u * kSubBlocks));
        if (!out.outside(p, 4u)) __stcs(p, __byte_perm(ta, tb, 0x6420));
    }
};

// Fused matrix-vector product: the 8 values are weights of one row of W (stored [rows, cols],
// cols a multiple of 256, so the 32 lanes of a step stay inside one row) and meet the 8
// matching entries of x of every token, staged in shared memory as fp16 token after token
// (tokens beyond the batch are zeros); products and sums in fp32, one accumulator per token.
// When the row ends the warp adds its lanes up.  A row that began and ended inside this
// chunk is complete: its sums are rounded to fp16 and stored.  A row that other chunks hold
// parts of gets the sums added to its fp32 accumulators, and the last chunk to do so rounds.
template <int B>
struct EmitDot {
    static constexpr bool kTwice = false;   // its values are added up: nothing wrong may pass
    uint32_t xaddr;       // shared-window address of x[0][col .. col + 8) for this lane's next group
    uint32_t xlane;       // the same at the start of a row
    uint32_t xstride;     // bytes from one token's x to the next
    uint32_t left;        // steps left in the current row
    uint32_t rs;          // steps per row (cols / 256)
    float acc[B];
    const GemvTensor* G;  // in shared memory
    uint32_t row;         // the current row
    uint32_t began_before;   // 1: the current row began in an earlier chunk
    uint32_t lane;
    uint32_t todo;        // groups left in the lane's sub-block
    __device__ __forceinline__ bool more() const { return todo != 0u; }

    __device__ __forceinline__ void flush(bool whole)
    {
#pragma unroll
        for (int b = 0; b < B; ++b) {
            float v = acc[b];
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
            if (lane == 0 && (uint32_t)b < G->batch) {
                const uint64_t at = (uint64_t)b * G->rows + row;
                if (whole) G->y[at] = __half_as_ushort(__float2half_rn(v));
                else atomicAdd(G->y32 + at, v);
            }
            acc[b] = 0.f;
        }
        if (!whole && lane == 0) row_part_done(G, row);
        ++row;
        began_before = 0u;
        left = rs;
        xaddr = xlane;
    }
    // acc += w.lo * x.lo, then acc += w.hi * x.hi: fp16 operands, fp32 sum, one rounding per step
    // (the product of two fp16 values is exact in fp32, so this is fmaf on the converted values).
    static __device__ __forceinline__ void fma2(float& acc, uint32_t w, uint32_t x)
    {
        asm("{\n\t"
            ".reg .b16 wl, wh, xl, xh;\n\t"
            "mov.b32 {wl, wh}, %1;\n\t"
            "mov.b32 {xl, xh}, %2;\n\t"
            "fma.rn.f32.f16 %0, wl, xl, %0;\n\t"
            "fma.rn.f32.f16 %0, wh, xh, %0;\n\t"
            "}"
            : "+f"(acc)
            : "r"(w), "r"(x));
    }
    __device__ __forceinline__ void operator()(uint4 w)
    {
#pragma unroll
        for (int b = 0; b < B; ++b) {
            const uint4 x = lds128(xaddr + (uint32_t)b * xstride);
            fma2(acc[b], w.x, x.x);
            fma2(acc[b], w.y, x.y);
            fma2(acc[b], w.z, x.z);
            fma2(acc[b], w.w, x.w);
        }
        xaddr += 512u;
        --todo;
        if (--left == 0u) flush(began_before == 0u);
    }
    __device__ __forceinline__ void finish()
    {
        if (left != rs) flush(false);     // the chunk ended inside a row
    }
};

// 8-bit alphabets, eight symbols per turn.  G = 2, 3 (as 3 + 3 + 2): groups of that many
// lookups, each checked.  G = 8: two groups of four under one check (the modes 4, 8 and 9 of
// the table build); if only the second failed it is repaired by itself, else both are done
// again one by one.  G = 16: all eight lookups on one view (at most 2 bit per symbol), done
// again as two fours if it fails.
template <int K, int G, class Emit>
__device__ __forceinline__ uint32_t rows_single(uint32_t start, uint32_t* status, LutKey key, Emit& emit)
{
    Cur r;
    cur_init(r, start);
    while (emit.more()) {
        uint32_t pk[4];
        bool again = false;
        if (G == 16) {
            uint4 v;
            uint32_t s;
            group8(r, key, v, s);
            pk[0] = v.x, pk[1] = v.y, pk[2] = v.z, pk[3] = v.w;
            if (__builtin_expect((s & 0xffe0u) != 0u, 0)) {
                cur_init(r, rewind_group(r, s));
                again = true;
            }
        }
        if (G == 8) {
            uint32_t s0, s1;
            group4(r, key, pk[0], pk[1], s0);
            group4(r, key, pk[2], pk[3], s1);
            if (__builtin_expect(((s0 | s1) & 0xffe0u) != 0u, 0)) {
                if ((s0 & 0xffe0u) == 0u) {
                    // the first four stand: only the second four are repaired
                    repair_quad<K>(r, status, key, s1, pk[2], pk[3]);
                } else {
                    // back over both: the position moved by s0 + s1, the words by one per flip of bit 5
                    const uint32_t p1 = r.pos - s1, p0 = p1 - s0;
                    const uint32_t steps = (((p0 ^ p1) >> 5) & 1u) + (((p1 ^ r.pos) >> 5) & 1u);
                    cur_init(r, (r.next - kCurBytes - 4u * steps) * 8u + (p0 & 31u));
                    again = true;
                }
            }
        }
        if (G == 8 || G == 16) {
            if (again) {
#pragma unroll
                for (int g = 0; g < 2; ++g) {
                    uint32_t s;
                    group4(r, key, pk[2 * g], pk[2 * g + 1], s);
                    if (__builtin_expect((s & 0xffe0u) != 0u, 0)) repair_quad<K>(r, status, key, s, pk[2 * g], pk[2 * g + 1]);
                }
            }
        } else if (G == 3) {
            // 3 + 3 + 2 under one check; what failed first is repaired, what came after it is done again
            uint32_t sa, sb, sc, a2, b0;
            group3<false>(r, key, pk[0], a2, sa);
            group3<true>(r, key, b0, pk[2], sb);
            group2(r, key, pk[3], sc);
            if (__builtin_expect(((sa | sb | sc) & 0xffe0u) != 0u, 0)) {
                const bool fa = (sa & 0xffe0u) != 0u;
                bool fb = (sb & 0xffe0u) != 0u;
                if (fa | fb) {
                    unwind_group(r, sc);
                    if (fa) {
                        unwind_group(r, sb);
                        repair_triple<K, false>(r, status, key, sa, pk[0], a2);
                        group3<true>(r, key, b0, pk[2], sb);
                        fb = (sb & 0xffe0u) != 0u;
                    }
                    if (fb) repair_triple<K, true>(r, status, key, sb, b0, pk[2]);
                    group2(r, key, pk[3], sc);
                }
                if ((sc & 0xffe0u) != 0u) repair_pair<K>(r, status, key, sc, pk[3]);
            }
            pk[1] = __byte_perm(a2, b0, 0x7632);
        } else {
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                uint32_t s;
                group2(r, key, pk[g], s);
                if (__builtin_expect((s & 0xffe0u) != 0u, 0)) repair_pair<K>(r, status, key, s, pk[g]);
            }
        }
        emit(make_uint4(pk[0], pk[1], pk[2], pk[3]));
        if (ENTRO_CHECK(smem_ok(r.next, 4u))) break;      // the next word the reader would pull in
    }
    return cur_bit_addr(r);
}

// 8-bit alphabets whose groups of four almost never fail, turns per chunk that come in N's,
// values that are stored: 8 N symbols, 2 N groups of four, under one check.  Each eight leave
// as soon as they are decoded (their registers are free for the next eight); if any of the
// groups failed, the eights from the first one with a failed group onwards are done again one
// group at a time and written again.
// kWide: every eight are one group of eight lookups on one view (streams of at most 2 bit per
// symbol) instead of two groups of four; a failure is repaired in fours all the same.
template <int K, int N, bool kWide, class Emit>
__device__ __forceinline__ uint32_t rows_multi(uint32_t start, uint32_t* status, LutKey key, Emit& emit)
{
    Cur r;
    cur_init(r, start);
    while (emit.more()) {
        uint32_t pk[4], s[2 * N], any = 0;
#pragma unroll
        for (int h = 0; h < N; ++h) {
            if (kWide) {
                uint4 v;
                group8(r, key, v, s[2 * h]);
                pk[0] = v.x, pk[1] = v.y, pk[2] = v.z, pk[3] = v.w;
                s[2 * h + 1] = 0u;
            } else {
                group4(r, key, pk[0], pk[1], s[2 * h]);
                group4(r, key, pk[2], pk[3], s[2 * h + 1]);
            }
            any |= s[2 * h] | s[2 * h + 1];
            if (h + 1 < N) emit(make_uint4(pk[0], pk[1], pk[2], pk[3]));
        }
        if (__builtin_expect((any & 0xffe0u) != 0u, 0)) {
            // the eights before the first one with a failed group stand; back over the groups from there
            // on: the position moved by the sum of their s, the words by one per flip of bit 5
            int h0 = 0;
#pragma unroll
            for (int h = N - 1; h >= 0; --h)
                if (((s[2 * h] | s[2 * h + 1]) & 0xffe0u) != 0u) h0 = h;
            uint32_t p = r.pos, steps = 0;
#pragma unroll
            for (int g = 2 * N - 1; g >= 0; --g) {
                if (g >= 2 * h0) {
                    const uint32_t before = p - s[g];
                    steps += ((before ^ p) >> 5) & 1u;
                    p = before;
                }
            }
            cur_init(r, (r.next - kCurBytes - 4u * steps) * 8u + (p & 31u));
            emit.back((uint32_t)(N - 1 - h0));
#pragma unroll 1
            for (int h = h0; h < N; ++h) {
#pragma unroll
                for (int g = 0; g < 2; ++g) {
                    uint32_t sg;
                    group4(r, key, pk[2 * g], pk[2 * g + 1], sg);
                    if (__builtin_expect((sg & 0xffe0u) != 0u, 0)) repair_quad<K>(r, status, key, sg, pk[2 * g], pk[2 * g + 1]);
                }
                if (h + 1 < N) emit(make_uint4(pk[0], pk[1], pk[2], pk[3]));
            }
        }
        emit(make_uint4(pk[0], pk[1], pk[2], pk[3]));
        if (ENTRO_CHECK(smem_ok(r.next, 4u))) break;      // the next word the reader would pull in
    }
    return cur_bit_addr(r);
}

// 4-bit alphabets: eight symbols per lookup.
template <int K, class Emit>
__device__ __forceinline__ uint32_t rows_oct(uint32_t start, uint32_t* status, Emit& emit)
{
    Win r;
    win_init<false>(r, (start >> 5) << 2, start & 31u);
    while (emit.more()) {
        win_refill<false>(r);
        const uint32_t idx = r.hi >> (32 - K);
        uint4 v = *reinterpret_cast<const uint4*>(smem + idx * 16u);
        const uint32_t n = *(smem + (16u << K) + idx);
        if (__builtin_expect(n == 0u, 0)) v = repair_oct<K>(r, status);
        else win_skip(r, n);
        emit(v);
    }
    return r.next * 8u - (uint32_t)win_valid_bits(r.k);
}

// The whole sub-block of a lane in the mode build_tables_kernel chose for the tensor;
// returns where the lane stands afterwards.
template <int K, class Emit>
__device__ __forceinline__ uint32_t rows_any(const DecodeAux* aux, uint32_t start, uint32_t* status, Emit& emit,
                                             uint32_t lane)
{
    const uint32_t mode = aux->mode;
    if (mode == 0u) return rows_oct<K>(start, status, emit);
    const LutKey key = lut_key(aux, lane);
    if constexpr (Emit::kTwice) {
        if (mode == 9u) return rows_multi<K, 2, false>(start, status, key, emit);
        if (mode == 17u) return rows_multi<K, 2, true>(start, status, key, emit);
        if (mode == 18u) return rows_multi<K, 4, true>(start, status, key, emit);
    }
    if (mode == 8u || mode == 9u || mode == 4u) return rows_single<K, 8>(start, status, key, emit);
    if (mode == 3u) return rows_single<K, 3>(start, status, key, emit);
    if (mode == 16u || mode == 17u || mode == 18u) return rows_single<K, 16>(start, status, key, emit);
    return rows_single<K, 2>(start, status, key, emit);
}

// What decode_start leaves for decode_finish: where this lane begins and must end.
struct Lane {
    uint32_t start, end;       // staged: shared-window bit addresses; general: bits before this lane's, and its count
    uint32_t kind;
};

// First half of decoding chunk r (its index slot is about to be reused): lane positions by
// a warp prefix sum over the sub-block lengths, checked against the offsets.
template <int K>
__device__ __forceinline__ Lane decode_start(const WarpCtx& cx, uint32_t* status, const Ready& r, uint32_t slot,
                                             uint32_t lane)
{
    Lane L;
    L.start = L.end = 0;
    L.kind = r.c == kNone ? (uint32_t)kSkip : r.kind();
    if (L.kind == kSkip) return L;
    const uint32_t pair = lds32(slot + (lane >> 1) * 4u);
    const uint32_t bits = (lane & 1u) ? pair >> 16 : pair & 0xffffu;
    // inclusive prefix sum over the lanes: a shuffle says by itself whether its source lane exists
    uint32_t incl = bits;
#define ENTRO_SCAN_STEP(d)                                     \
    "shfl.sync.up.b32 t|p, %0, " #d ", 0, 0xffffffff;\n\t"      \
    "@p add.u32 %0, %0, t;\n\t"
    asm volatile("{\n\t.reg .pred p;\n\t.reg .b32 t;\n\t" ENTRO_SCAN_STEP(1) ENTRO_SCAN_STEP(2) ENTRO_SCAN_STEP(4)
                     ENTRO_SCAN_STEP(8) ENTRO_SCAN_STEP(16) "}"
                 : "+r"(incl));
#undef ENTRO_SCAN_STEP
    const uint32_t total = __shfl_sync(0xffffffffu, incl, 31);
    // (prepare has checked that the chunk is shorter than 2^21 bits: the low words decide)
    const uint32_t off0 = lds32(slot + 64u), off1 = lds32(slot + 72u);
    if (off1 - off0 != total) {                 // the recorded lengths do not add up to the chunk
        if (lane == 0) atomicOr(status, kStatCorrupt);
        L.kind = kSkip;
        return L;
    }
    const uint32_t excl = incl - bits;
    if (L.kind == kGeneral) {
        L.start = excl;
        L.end = bits;
    } else {
        // (off0 & 127: the chunk's first bit behind the 16-byte boundary the copy started at)
        L.start = (cx.stage_addr + r.at()) * 8u + (off0 & 127u) + excl;
        L.end = L.start + bits;
    }
    return L;
}

template <int K, int kSink>
__device__ __forceinline__ void decode_finish(WarpCtx& cx, uint32_t* status, Ready& r, Lane L, uint32_t lane,
                                              uint32_t stage_bytes)
{
    constexpr int kBatch = kGemvBatchOf<kSink>;
    constexpr bool kGemv = kBatch > 0;
    if (L.kind == kSkip) return;
    const DevTensor& T = *tensor_ptr<K>();
    const GemvTensor* G = kGemv ? gemv_ptr<K>() : nullptr;
    if (L.kind == kStaged) {
        if (!r.issued()) issue_copy(cx, T, r, (T.offsets[r.c] >> 3) & ~15ull, lane, stage_bytes);
        bool ok = mbar_wait(cx.bar + 8u * (r.ticket() & 1u), (r.ticket() >> 1) & 1u);
        ok = __all_sync(0xffffffffu, ok);
        if (!ok) {
            if (lane == 0) atomicOr(status, kStatTimeout);
            cx.state |= 1u << 31;
            // fall back to global memory: bits of the chunk before this lane's, and this lane's count
            const uint32_t first = __shfl_sync(0xffffffffu, L.start, 0);
            L.kind = kGeneral;
            L.end -= L.start;
            L.start -= first;
        }
    }
    if (L.kind == kGeneral) {
        decode_chunk_general<kBatch>(aux_ptr<K>(), status, T, G, kSink, r.c, L.start, L.end, lane);
        return;
    }
    const uint32_t turns = aux_ptr<K>()->turns;     // groups of 8 symbols per lane (staged chunks have whole groups only)
    uint32_t stood;            // where the lane stands after its sub-block
    if (kGemv) {
        // the chunk starts gs0 steps of 256 weights into the matrix; a row is rs steps long
        const uint32_t rs = G->cols >> 8;
        const uint32_t gs0 = (uint32_t)(((uint64_t)r.c * T.chunk_symbols) >> 8);
        const uint32_t row0 = gs0 / rs, k0 = gs0 - row0 * rs;
        EmitDot<kGemv ? kBatch : 1> em;
        em.lane = lane;
        em.rs = rs;
        em.left = rs - k0;
        em.xlane = kSmemBase + kGemvX<K> + lane * 16u;
        em.xaddr = em.xlane + k0 * 512u;
        em.xstride = G->cols * 2u;
#pragma unroll
        for (int b = 0; b < (kGemv ? kBatch : 1); ++b) em.acc[b] = 0.f;
        em.G = G;
        em.row = row0;
        em.began_before = k0 != 0u;
        em.todo = turns;
        stood = rows_any<K>(aux_ptr<K>(), L.start, status, em, lane);
        em.finish();
    } else if (kSink == kSinkBytes) {
        EmitBytes em;
        em.out.start(reinterpret_cast<uint8_t*>(T.out) + (uint64_t)r.c * T.chunk_symbols + lane * 8u, turns, 8u * kSubBlocks);
        em.out.bounds(T.out, T.n);
        stood = rows_any<K>(aux_ptr<K>(), L.start, status, em, lane);
    } else if (kSink == kSinkNibbles) {
        EmitNibbles em;
        em.out.start(reinterpret_cast<uint8_t*>(T.out) + (((uint64_t)r.c * T.chunk_symbols) >> 1) + lane * 4u, turns,
                     4u * kSubBlocks);
        em.out.bounds(T.out, (T.n + 1u) >> 1);
        stood = rows_any<K>(aux_ptr<K>(), L.start, status, em, lane);
    } else {
        EmitStore em;
        em.out.start(T.out + (uint64_t)r.c * T.chunk_symbols + lane * 8u, turns, 16u * kSubBlocks);
        em.out.bounds(T.out, T.n * 2u);
        stood = rows_any<K>(aux_ptr<K>(), L.start, status, em, lane);
        em.finish();
    }
    // the lane must stand exactly at the end of its sub-block
    if (stood != L.end) atomicOr(status, kStatCorrupt);
    __syncwarp();   // all lanes are done with these bytes before the ring reuses them
}

}  // namespace
}  // namespace entro
