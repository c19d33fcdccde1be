// Bit readers and table lookups of the decode kernel: the 64-bit window, the three-word
// reader of the grouped lookups, the hand-scheduled groups and their repairs.
// Included by entro_decode.cu only.
#pragma once

#include "entro_decode_tables.cuh"

namespace entro {
namespace {

// ------------------------------------------------------------------ bit reader

// 64-bit window, left-justified, zeros below the valid bits.  `k` is 32 minus the number
// of valid bits, kept modulo 2^16 in the low half of the register (the high half may hold
// anything): negative (bit 15 set) while more than 32 bits are valid, else the left shift
// that puts the next word behind the valid bits.  With kInv the window holds the
// complement of the stream bits (what the exponent-indexed table wants).
struct Win {
    uint32_t hi, lo;
    uint32_t k;
    uint32_t next;            // shared-window address of the next word to pull in
};

// Window over the bits that start `bit_pos` bits after shared-window address `base`.
template <bool kInv>
__device__ __forceinline__ void win_init(Win& r, uint32_t base, uint32_t bit_pos)
{
    const uint32_t p = base + ((bit_pos >> 5) << 2);
    const uint32_t bit = bit_pos & 31u;
    uint32_t w0 = lds32(p), w1 = lds32(p + 4);
    if (kInv) {
        w0 = ~w0;
        w1 = ~w1;
    }
    r.hi = __funnelshift_l(w1, w0, bit);
    r.lo = w1 << bit;
    r.k = bit - 32u;          // 64 - bit valid bits
    r.next = p + 8;
}

// Top up to more than 32 valid bits.  With 32 or fewer the low word is empty.
template <bool kInv>
__device__ __forceinline__ void win_refill(Win& r)
{
    if (!(r.k & 0x8000u)) {
        uint32_t w = lds32(r.next);
        r.next += 4;
        if (kInv) w = ~w;
        r.hi |= __funnelshift_l(w, 0u, r.k);      // w >> (32 - k), nothing for k = 0
        r.lo = __funnelshift_l(0u, w, r.k);       // w << k
        r.k -= 32u;
    }
}

// Drop n bits, 0 <= n <= 31 in the low five bits of n; n's low half is the true count.
__device__ __forceinline__ void win_skip(Win& r, uint32_t n)
{
    r.hi = __funnelshift_l(r.lo, r.hi, n);
    r.lo = __funnelshift_l(0u, r.lo, n);
    r.k += n;
}

// Drop n bits, 0 <= n <= 32.
__device__ __forceinline__ void win_skip_any(Win& r, uint32_t n)
{
    r.hi = __funnelshift_lc(r.lo, r.hi, n);
    r.lo = __funnelshift_lc(0u, r.lo, n);
    r.k += n;
}

__device__ __forceinline__ int win_valid_bits(uint32_t k) { return 32 - (int)(short)(k & 0xffffu); }

// The same over global memory, word by word, for chunks that are not staged.
struct GlobalWin {
    uint32_t hi, lo;
    int nb;
    uint32_t next;
    const uint32_t* words;
    uint64_t count;           // words readable from `words`
    __device__ __forceinline__ uint32_t get(uint32_t i) const { return i < count ? __ldg(words + i) : 0u; }
};

__device__ __forceinline__ void gwin_refill(GlobalWin& r)
{
    if (r.nb <= 32) {
        uint32_t w = r.get(r.next);
        r.next++;
        r.hi |= __funnelshift_rc(w, 0u, (uint32_t)r.nb);
        r.lo = __funnelshift_lc(0u, w, (uint32_t)(32 - r.nb));
        r.nb += 32;
    }
}

// ------------------------------------------------------------------ lookups

// How a lane addresses its copy of the exponent-indexed table (which starts at the
// beginning of shared memory, cell-major): byte offset = ((float bits >> 12) & mask) | lane.
// 32 << m cells, 32 >> (m - 4) copies, cells (128 >> (m - 4)) bytes apart: always 64 KB, and the
// cell index (float bits 27 .. 23 - m) always lands on its byte offset by a shift of 12.
struct LutKey {
    uint32_t mask, lane;
};
__device__ __forceinline__ LutKey lut_key(const DecodeAux* aux, uint32_t lane)
{
    LutKey k;
    k.mask = aux->key_mask;
    k.lane = (lane & aux->key_lane_mask) * 4u;
    return k;
}

// Cell of the exponent-indexed table for an inverted window, in this lane's copy.
__device__ __forceinline__ uint32_t exp_lookup(LutKey key, uint32_t inv_window)
{
    const uint32_t fb = __float_as_uint(__uint2float_rz(inv_window));
    const uint32_t a = ((fb >> 12) & key.mask) | key.lane;
    if (ENTRO_CHECK(a < 4u * (uint32_t)kExpEntriesMax && (a & 3u) == 0u)) return kEscLen;
    return *reinterpret_cast<const uint32_t*>(smem + a);
}

// One symbol from a full 32-bit window (true stream bits) by the canonical ranges; a pattern
// that is no codeword is flagged and dropped as a single bit.  -> value << 16 | length.
__device__ __forceinline__ uint32_t decode_by_range(const DecodeAux* aux, uint32_t window, uint32_t* status)
{
    uint32_t len;
    uint32_t sym = range_decode(*aux, window, aux->max_len, len);
    if (len == 0) {
        atomicOr(status, kStatCorrupt);
        return 1u;
    }
    return ((uint32_t)aux->val[sym] << 16) | len;
}

// Reader of the grouped lookups of 8-bit alphabets: three consecutive stream words
// (complemented) in registers and a bit position whose low five bits say where in w0 the
// next code starts.  Only those five bits and bit 5 (has a word boundary been crossed?) are
// ever used, so the upper bits of pos may hold anything.  A group reads w0 and w1 only; w2
// is held ahead so that the word read from shared memory when a boundary is crossed is not
// needed before the boundary after it (the read is off the chain from group to group).
struct Cur {
    uint32_t w0, w1, w2;
    uint32_t pos;
    uint32_t next;            // shared-window address of the word after w2
};
constexpr uint32_t kCurBytes = 12;   // bytes from w0's address to next

__device__ __forceinline__ void cur_init(Cur& c, uint32_t bit_addr)
{
    const uint32_t a = (bit_addr >> 5) << 2;
    c.w0 = ~lds32(a);
    c.w1 = ~lds32(a + 4);
    c.w2 = ~lds32(a + 8);
    c.next = a + kCurBytes;
    c.pos = bit_addr;
}

// Shared-window bit address the reader stands at.
__device__ __forceinline__ uint32_t cur_bit_addr(const Cur& c) { return (c.next - kCurBytes) * 8u + (c.pos & 31u); }

// One group of lookups, hand-scheduled.  The group sees the 32 bits that start at the
// reader's position (one funnel shift of the first two words) and nothing behind them: a lookup
// reads them shifted left by the lengths found before it (a funnel shift uses the low five
// bits of its count), zeros moving in from the right.  Those
// zeros cannot mislead a lookup whose code ends inside the 32 bits: a cell is resolved only
// if every window that maps to it begins with the same code, whatever follows.  s is the sum
// of the G entries: the group stands iff (s & 0xffe0) == 0, that is, every cell was resolved
// (an unresolved one adds 64) and fewer than 32 bits were used, so all codes did end inside
// the 32 bits.  Then the position moves on by s and, if that crosses into the next word
// (bit 5 of the position flips), the words move up by one and a new third word is pulled
// in, predicated.
// If the group does not stand the caller repairs it from rewind_group, which needs only
// pos, next and s.
// Checked build: the cell's byte offset must lie inside the 64 KB of the table, else the
// violation is counted and cell 0 is read instead.
#ifdef ENTRO_CHECKED
#define ENTRO_CELL_CHECK_AT(counter)                 \
    "setp.gt.u32 q, a, 65532;\n\t"                    \
    "@q red.global.add.u32 [" counter "], 1;\n\t"     \
    "@q mov.b32 a, 0;\n\t"
#define ENTRO_CELL_CHECK ENTRO_CELL_CHECK_AT("%10")
#define ENTRO_CHECK_REGS ".reg .pred q;\n\t"
#define ENTRO_CHECK_ARG , "l"(&g_check_violations)
#else
#define ENTRO_CELL_CHECK_AT(counter)
#define ENTRO_CELL_CHECK
#define ENTRO_CHECK_REGS
#define ENTRO_CHECK_ARG
#endif
#define ENTRO_LOOKUP(dst, win)                       \
    "cvt.rz.f32.u32 f, " win ";\n\t"                  \
    "mov.b32 a, f;\n\t"                               \
    "shr.u32 a, a, 12;\n\t"                           \
    "lop3.b32 a, a, %9, %8, 0xEA;\n\t" ENTRO_CELL_CHECK \
    "ld.shared.b32 " dst ", [a+1024];\n\t"
#define ENTRO_OPEN                                   \
    "shf.l.wrap.b32 h, %1, %0, %2;\n\t"
#define ENTRO_MOVE_ON                                \
    "add.u32 t, %2, %6;\n\t"                          \
    "xor.b32 a, t, %2;\n\t"                           \
    "mov.b32 %2, t;\n\t"                              \
    "and.b32 a, a, 32;\n\t"                           \
    "setp.ne.u32 p, a, 0;\n\t"                        \
    "@p mov.b32 %0, %1;\n\t"                          \
    "@p mov.b32 %1, %7;\n\t"                          \
    "@p ld.shared.b32 t, [%3];\n\t"                   \
    "@p add.u32 %3, %3, 4;\n\t"                       \
    "@p not.b32 %7, t;\n\t"

__device__ __forceinline__ void group4(Cur& c, LutKey key, uint32_t& pk0, uint32_t& pk1, uint32_t& s)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t" ENTRO_CHECK_REGS
        ".reg .b32 t, w, a, h, e0, e1, e2, e3;\n\t"
        ".reg .f32 f;\n\t" ENTRO_OPEN ENTRO_LOOKUP("e0", "h")
        "shf.l.wrap.b32 w, 0, h, e0;\n\t" ENTRO_LOOKUP("e1", "w")
        "add.u32 %6, e0, e1;\n\t"
        "shf.l.wrap.b32 w, 0, h, %6;\n\t" ENTRO_LOOKUP("e2", "w")
        "add.u32 %6, %6, e2;\n\t"
        "shf.l.wrap.b32 w, 0, h, %6;\n\t" ENTRO_LOOKUP("e3", "w")
        "add.u32 %6, %6, e3;\n\t"
        "prmt.b32 %4, e0, e1, 0x7632;\n\t"
        "prmt.b32 %5, e2, e3, 0x7632;\n\t" ENTRO_MOVE_ON "}"
        : "+r"(c.w0), "+r"(c.w1), "+r"(c.pos), "+r"(c.next), "=&r"(pk0), "=&r"(pk1), "=&r"(s), "+r"(c.w2)
        : "r"(key.lane), "r"(key.mask) ENTRO_CHECK_ARG);
}

__device__ __forceinline__ void group2(Cur& c, LutKey key, uint32_t& pk0, uint32_t& s)
{
    __attribute__((unused)) uint32_t unused;   // operand slot of the second pair, which a group of two does not have
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t" ENTRO_CHECK_REGS
        ".reg .b32 t, w, a, h, e0, e1;\n\t"
        ".reg .f32 f;\n\t" ENTRO_OPEN ENTRO_LOOKUP("e0", "h")
        "shf.l.wrap.b32 w, 0, h, e0;\n\t" ENTRO_LOOKUP("e1", "w")
        "add.u32 %6, e0, e1;\n\t"
        "prmt.b32 %4, e0, e1, 0x7632;\n\t"
        "mov.b32 %5, 0;\n\t" ENTRO_MOVE_ON "}"
        : "+r"(c.w0), "+r"(c.w1), "+r"(c.pos), "+r"(c.next), "=&r"(pk0), "=&r"(unused), "=&r"(s), "+r"(c.w2)
        : "r"(key.lane), "r"(key.mask) ENTRO_CHECK_ARG);
}
// Three lookups, for the streams whose groups of four would too often need 32 bits or more.
// Eight symbols go out as 3 + 3 + 2, so the pairs of values straddle the groups: with kTail
// false, first = the pair (v0, v1) and second = the third entry as it is; with kTail true,
// first = the first entry as it is and second = the pair (v1, v2).
template <bool kTail>
__device__ __forceinline__ void group3(Cur& c, LutKey key, uint32_t& first, uint32_t& second, uint32_t& s)
{
    if (!kTail)
        asm volatile(
            "{\n\t"
            ".reg .pred p;\n\t" ENTRO_CHECK_REGS
            ".reg .b32 t, w, a, h, e0, e1;\n\t"
            ".reg .f32 f;\n\t" ENTRO_OPEN ENTRO_LOOKUP("e0", "h")
            "shf.l.wrap.b32 w, 0, h, e0;\n\t" ENTRO_LOOKUP("e1", "w")
            "shf.l.wrap.b32 w, 0, w, e1;\n\t" ENTRO_LOOKUP("%5", "w")
            "add.u32 %6, e0, e1;\n\t"
            "add.u32 %6, %6, %5;\n\t"
            "prmt.b32 %4, e0, e1, 0x7632;\n\t" ENTRO_MOVE_ON "}"
            : "+r"(c.w0), "+r"(c.w1), "+r"(c.pos), "+r"(c.next), "=&r"(first), "=&r"(second), "=&r"(s), "+r"(c.w2)
            : "r"(key.lane), "r"(key.mask) ENTRO_CHECK_ARG);
    else
        asm volatile(
            "{\n\t"
            ".reg .pred p;\n\t" ENTRO_CHECK_REGS
            ".reg .b32 t, w, a, h, e1, e2;\n\t"
            ".reg .f32 f;\n\t" ENTRO_OPEN ENTRO_LOOKUP("%4", "h")
            "shf.l.wrap.b32 w, 0, h, %4;\n\t" ENTRO_LOOKUP("e1", "w")
            "shf.l.wrap.b32 w, 0, w, e1;\n\t" ENTRO_LOOKUP("e2", "w")
            "add.u32 %6, %4, e1;\n\t"
            "add.u32 %6, %6, e2;\n\t"
            "prmt.b32 %5, e1, e2, 0x7632;\n\t" ENTRO_MOVE_ON "}"
            : "+r"(c.w0), "+r"(c.w1), "+r"(c.pos), "+r"(c.next), "=&r"(first), "=&r"(second), "=&r"(s), "+r"(c.w2)
            : "r"(key.lane), "r"(key.mask) ENTRO_CHECK_ARG);
}
// Eight lookups on one view, for streams of so few bits per symbol (at most 2) that eight
// codes almost always fit 32 bits: 4-bit alphabets beyond the reach of the eight-symbol table.
#define ENTRO_LOOKUP8(dst, win)                      \
    "cvt.rz.f32.u32 f, " win ";\n\t"                  \
    "mov.b32 a, f;\n\t"                               \
    "shr.u32 a, a, 12;\n\t"                           \
    "lop3.b32 a, a, %11, %10, 0xEA;\n\t" ENTRO_CELL_CHECK_AT("%12") \
    "ld.shared.b32 " dst ", [a+1024];\n\t"
#define ENTRO_NEXT8(e)                               \
    "add.u32 %6, %6, " e ";\n\t"                      \
    "shf.l.wrap.b32 w, 0, h, %6;\n\t"
__device__ __forceinline__ void group8(Cur& c, LutKey key, uint4& pk, uint32_t& s)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t" ENTRO_CHECK_REGS
        ".reg .b32 t, w, a, h, e0, e1, e2, e3, e4, e5, e6, e7;\n\t"
        ".reg .f32 f;\n\t" ENTRO_OPEN ENTRO_LOOKUP8("e0", "h")
        "shf.l.wrap.b32 w, 0, h, e0;\n\t" ENTRO_LOOKUP8("e1", "w")
        "add.u32 %6, e0, e1;\n\t"
        "shf.l.wrap.b32 w, 0, h, %6;\n\t" ENTRO_LOOKUP8("e2", "w") ENTRO_NEXT8("e2") ENTRO_LOOKUP8("e3", "w")
        ENTRO_NEXT8("e3") ENTRO_LOOKUP8("e4", "w") ENTRO_NEXT8("e4") ENTRO_LOOKUP8("e5", "w")
        ENTRO_NEXT8("e5") ENTRO_LOOKUP8("e6", "w") ENTRO_NEXT8("e6") ENTRO_LOOKUP8("e7", "w")
        "add.u32 %6, %6, e7;\n\t"
        "prmt.b32 %4, e0, e1, 0x7632;\n\t"
        "prmt.b32 %5, e2, e3, 0x7632;\n\t"
        "prmt.b32 %8, e4, e5, 0x7632;\n\t"
        "prmt.b32 %9, e6, e7, 0x7632;\n\t" ENTRO_MOVE_ON "}"
        : "+r"(c.w0), "+r"(c.w1), "+r"(c.pos), "+r"(c.next), "=&r"(pk.x), "=&r"(pk.y), "=&r"(s), "+r"(c.w2), "=&r"(pk.z),
          "=&r"(pk.w)
        : "r"(key.lane), "r"(key.mask) ENTRO_CHECK_ARG);
}
#undef ENTRO_LOOKUP8
#undef ENTRO_NEXT8
#undef ENTRO_LOOKUP
#undef ENTRO_CELL_CHECK
#undef ENTRO_CELL_CHECK_AT
#undef ENTRO_CHECK_REGS
#undef ENTRO_CHECK_ARG
#undef ENTRO_OPEN
#undef ENTRO_MOVE_ON

// The next symbol by itself, any code length: refill, one exponent-indexed lookup (this
// lane's copy for 8-bit alphabets, the single copy behind the eight-symbol tables for 4-bit
// ones), the canonical ranges if the cell is unresolved.  -> value << 16 | length.
template <int K, bool kOct>
__device__ __forceinline__ uint32_t next_symbol(Win& r, uint32_t* status, LutKey key)
{
    win_refill<!kOct>(r);
    const uint32_t inv = kOct ? ~r.hi : r.hi;
    uint32_t e;
    if (kOct) {
        const uint32_t cell = (__float_as_uint(__uint2float_rz(inv)) >> (23 - kExpBitsMin)) & (uint32_t)(kExpEntriesMin - 1);
        e = *reinterpret_cast<const uint32_t*>(smem + (17u << K) + cell * 4u);
    } else {
        e = exp_lookup(key, inv);
    }
    if ((e & 0xffffu) > 32u) e = decode_by_range(reinterpret_cast<const DecodeAux*>(smem + lut_bytes(K)), ~inv, status);
    win_skip_any(r, e & 0xffffu);
    return e;
}

// Where the reader stood before a group that did not stand: the position moved on by
// exactly s (modulo 2^16), and the words moved on by one iff bit 5 of the position flipped.
__device__ __forceinline__ uint32_t rewind_group(const Cur& c, uint32_t s)
{
    const uint32_t before = c.pos - s;
    const uint32_t crossed = ((before ^ c.pos) >> 5) & 1u;
    return (c.next - kCurBytes - 4u * crossed) * 8u + (before & 31u);
}

// Takes the reader's position and word address back over a group that moved it on by s (the
// words themselves stay as they are: whoever repairs from here opens them anew).
__device__ __forceinline__ void unwind_group(Cur& c, uint32_t s)
{
    const uint32_t before = c.pos - s;
    c.next -= 4u * (((before ^ c.pos) >> 5) & 1u);
    c.pos = before;
}

// Repair of a group of two symbols that did not stand (kept inline: a call here would park
// the caller's registers in local memory, which misses the small L1 left beside 228 KB of
// shared memory): the symbols one by one, any code length, with the general reader.
template <int K>
__device__ __forceinline__ void repair_pair(Cur& c, uint32_t* status, LutKey key, uint32_t s, uint32_t& pk)
{
    const uint32_t at = rewind_group(c, s);
    Win r;
    win_init<true>(r, (at >> 5) << 2, at & 31u);
    const uint32_t e0 = next_symbol<K, false>(r, status, key);
    const uint32_t e1 = next_symbol<K, false>(r, status, key);
    pk = __byte_perm(e0, e1, 0x7632);
    cur_init(c, r.next * 8u - (uint32_t)win_valid_bits(r.k));
}

// The same for a group of three (rare by the choice of the group size).
template <int K, bool kTail>
__device__ __forceinline__ void repair_triple(Cur& c, uint32_t* status, LutKey key, uint32_t s, uint32_t& first,
                                              uint32_t& second)
{
    const uint32_t at = rewind_group(c, s);
    Win r;
    win_init<true>(r, (at >> 5) << 2, at & 31u);
    const uint32_t e0 = next_symbol<K, false>(r, status, key);
    const uint32_t e1 = next_symbol<K, false>(r, status, key);
    const uint32_t e2 = next_symbol<K, false>(r, status, key);
    first = kTail ? e0 : __byte_perm(e0, e1, 0x7632);
    second = kTail ? __byte_perm(e1, e2, 0x7632) : e2;
    cur_init(c, r.next * 8u - (uint32_t)win_valid_bits(r.k));
}

// Repair of a group of four: almost always it merely used 32 bits or more, so two groups of
// two stand; each of those falls back to repair_pair.
template <int K>
__device__ __forceinline__ void repair_quad(Cur& c, uint32_t* status, LutKey key, uint32_t s, uint32_t& pk0, uint32_t& pk1)
{
    cur_init(c, rewind_group(c, s));
    uint32_t s2;
    group2(c, key, pk0, s2);
    if (__builtin_expect((s2 & 0xffe0u) != 0u, 0)) repair_pair<K>(c, status, key, s2, pk0);
    group2(c, key, pk1, s2);
    if (__builtin_expect((s2 & 0xffe0u) != 0u, 0)) repair_pair<K>(c, status, key, s2, pk1);
}

// Eight symbols of a 4-bit alphabet whose codes do not fit the table's window.
template <int K>
__device__ __forceinline__ uint4 repair_oct(Win& r, uint32_t* status)
{
    uint32_t h[8];
#pragma unroll
    for (int k = 0; k < 8; ++k) h[k] = next_symbol<K, true>(r, status, LutKey{0u, 0u});
    return make_uint4(__byte_perm(h[0], h[1], 0x7632), __byte_perm(h[2], h[3], 0x7632), __byte_perm(h[4], h[5], 0x7632),
                      __byte_perm(h[6], h[7], 0x7632));
}

}  // namespace
}  // namespace entro
