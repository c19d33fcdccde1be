// Parallel Huffman decode fused with dequantisation to fp16 (Section 3, "Segmentation for
// parallel Huffman decoding"; Eq. 1 inverted).
//
// Work split: a chunk (one segment) is decoded by one warp, each lane owning one of the
// chunk's 32 sub-blocks.  The lanes' start positions come from a warp prefix sum over the
// sub-block bit lengths stored in the index.  A persistent grid pulls work items (runs of
// chunks of one tensor) from a global counter; the warps of a CTA share out an item's
// chunks through a shared-memory counter.  Every warp runs a three-deep pipeline: while it
// decodes chunk i, the bytes of chunk i + 1 are arriving in its shared-memory ring through
// one bulk asynchronous copy, and the index entries of chunk i + 2 are on their way into
// registers.  Lanes walk their bits with lookup tables whose entries already hold the
// dequantised fp16 values.  A sub-block is the chunk's 8-symbol groups l, l + 32, ..., so
// when every lane has decoded one group the warp's 32 16-byte stores cover 512
// contiguous bytes: four full lines per store instruction, no staging of the output.
//
// Tables per tensor (built by build_tables_kernel, copied into shared memory per CTA):
//   alphabets > 16 symbols, one symbol per lookup.  Canonical codes grow longer towards the
//     all-ones end of the code space, so the table is indexed like a floating-point number:
//     by the count of leading one bits of the window and the m bits after the first zero.
//     Converting the inverted window to float yields exactly that index (exponent | top
//     mantissa bits) in one instruction, and 32 << m cells resolve every code whose length
//     is at most leading ones + 1 + m - on bell-shaped histograms all of them, where a
//     direct table of the same size would miss the tail.  m = 4 when that already covers
//     the code (peaked, heavy-tailed histograms): the shared-memory copy is then replicated
//     32 times, cell-major, so lane l only ever touches bank l and no lookup conflicts,
//     whatever the data.  Flatter histograms get a larger m, up to 9, in the same 64 KB:
//     every extra bit halves the number of copies (16 copies: lanes l and l + 16 share one,
//     at most two wavefronts per lookup; ... ; one copy at m = 9).
//   alphabets <= 16 symbols, eight symbols per lookup: the next K bits index a table of
//     16-byte entries (eight fp16 values) and a byte table (bits used, 0 = no eight whole
//     codes in K bits); one unreplicated copy of the exponent-indexed table serves the
//     symbol-by-symbol repair of such windows.
//   aux   canonical ranges per length, for whatever the tables do not resolve.
#include <cuda_fp16.h>

#include "entro_internal.h"

namespace entro {
namespace {

extern __shared__ __align__(1024) unsigned char smem[];

constexpr uint32_t kNone = 0xffffffffu;
constexpr uint32_t kWaitTries = 1u << 16;  // bound on polling a bulk copy (each try may suspend)
constexpr uint32_t kEscLen = 0x40u;        // length field of a cell the table cannot resolve
constexpr uint32_t kOverRead = 2064;       // a lane fed garbage may read this far past its chunk's bytes
// Address of dynamic shared memory in the shared window on sm_100 (the first KiB of the
// window is the driver's).  The hand-written lookups address the tables as [offset + 1024];
// the kernel checks the assumption before it does anything else.
constexpr uint32_t kSmemBase = 1024;
static_assert(kExpBitsMin == 4 && kExpBitsMax == 9,
              "the lookups shift the float bits by 12 whatever m is because cells * copies * 4 bytes = 64 KB");

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
// 32-bit word at a shared-window address.
__device__ __forceinline__ uint32_t lds32(uint32_t addr)
{
    uint32_t v;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

// Shared-memory bytes of the lookup tables for a K-bit eight-symbol table.
__host__ __device__ constexpr uint32_t lut_bytes(int K)
{
    return (17u << K) + 4u * kExpEntriesMin > 65536u ? (17u << K) + 4u * kExpEntriesMin : 65536u;
}

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
// The grid is (tensors, kTableSlices): every block of a tensor works out the small things
// for itself and fills its share of the tables' entries.
constexpr unsigned kTableSlices = 8;
__global__ void __launch_bounds__(256) build_tables_kernel(const DevTensor* __restrict__ tensors, int lut_bits,
                                                           TensorTables* __restrict__ tables,
                                                           uint32_t* __restrict__ control,
                                                           const GemvTensor* __restrict__ gemv)
{
    __shared__ DecodeAux aux;
    __shared__ uint32_t count[ENTRO_MAX_CODE_LEN + 1];
    __shared__ uint8_t len[ENTRO_MAX_SYMBOLS];
    __shared__ float need_mass[16];   // probability mass (by 2^-length) of the codes that need j bits behind their first zero
    const int t = blockIdx.x;
    const int tid = threadIdx.x;
    const DevTensor& T = tensors[t];
    TensorTables& out = tables[t];
    const uint32_t first = blockIdx.y * 256u + (uint32_t)tid, stride = gridDim.y * 256u;   // this thread's entries
    if (t == 0 && first == 0) control[0] = 0;   // work counter of the decode kernel that follows
    if (gemv) {                                 // and the fp32 sums of the fused matrix-vector products
        float* y32 = gemv[t].y32;
        const uint32_t n = gemv[t].rows * gemv[t].batch;
        for (uint32_t i = first; i < n; i += stride) y32[i] = 0.f;
    }
    if (tid <= ENTRO_MAX_CODE_LEN) count[tid] = 0;
    len[tid] = (uint32_t)tid < T.nsym ? T.len[tid] : 0;
    __syncthreads();
    const uint32_t l = len[tid];
    if (l) atomicAdd(&count[l], 1u);
    __syncthreads();
    if (tid == 0) {
        unsigned long long code = 0;   // reaches 2^32 after the last length of a complete code
        uint32_t off = 0, max_len = 0;
        // bits per symbol of this tensor's stream, from the index (a wrong index can only pick a slower mode)
        const float mean_len = (float)T.offsets[T.n_chunks] / (float)T.n;
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
        // eight symbols per lookup pay off while eight codes usually fit the table's window
        aux.oct = (T.nsym <= 16 && mean_len * 8.f <= (float)lut_bits - 1.5f) ? 1u : 0u;
        aux.group = 2u;            // decided below, from the chance that a group needs 32 bits or more
        aux.expm = (uint32_t)kExpBitsMin;
        for (int j = 0; j < 16; ++j) need_mass[j] = 0.f;
    }
    __syncthreads();
    if (l) {
        uint32_t rank = 0;
        for (int k = 0; k < tid; ++k) rank += (len[k] == l);
        aux.sorted[aux.offset[l] + rank] = (uint8_t)tid;
        // how many bits behind the first zero does a table need to resolve this symbol's code?
        // It has r leading ones, so l - r - 1 (none if the code is all ones).
        const uint32_t left = (aux.first_code[l] + rank) << (32u - l);
        uint32_t r = (uint32_t)__clz((int)~left);
        if (r > l) r = l;
        const uint32_t need = l > r + 1u ? l - r - 1u : 0u;
        atomicAdd(&need_mass[need < 15u ? need : 15u], exp2f(-(float)l));
    }
    __syncthreads();
    // Lookups per group: a group stands only if its codes use fewer than 32 bits together.
    // With 2^-length for the chance of a symbol, fail[g] = chance that g lengths sum to 32 or
    // more, by repeated convolution of the length distribution (bin 32 collects the rest).
    {
        __shared__ float by_len[33], dist[2][33], fail[5];
        if (tid <= 32) {
            by_len[tid] = tid ? (float)count[tid] * exp2f(-(float)tid) : 0.f;
            dist[0][tid] = tid == 0 ? 1.f : 0.f;
        }
        __syncthreads();
        for (int g = 1; g <= 4; ++g) {
            const float* in = dist[(g - 1) & 1];
            float* o = dist[g & 1];
            if (tid < 32) {
                float v = 0.f;
                for (int j = 0; j <= tid; ++j) v += in[j] * by_len[tid - j];
                o[tid] = v;
            }
            __syncthreads();
            if (tid == 0) {
                float in_range = 0.f;
                for (int j = 0; j < 32; ++j) in_range += o[j];
                fail[g] = fmaxf(1.f - in_range, 0.f);
                o[32] = 0.f;
            }
            __syncthreads();
        }
        if (tid == 0) {
            const float mean_len = (float)T.offsets[T.n_chunks] / (float)T.n;   // guards against a codebook that does not fit the data
            // a failing lane stalls its warp: the limits keep the warp's failures to a few per cent
            if (fail[4] < 3e-4f && mean_len <= 4.0f) aux.group = 8u;        // two groups of four under one check
            else if (fail[4] < 3e-3f && mean_len <= 5.2f) aux.group = 4u;
            else if (fail[3] < 2.4e-3f && mean_len <= 8.5f) aux.group = 3u;
        }
    }
    __syncthreads();
    if (tid == 0 && !aux.oct) {
        // the smallest table that leaves less than 6e-5 of the symbols to the repair path
        float open = 0.f;
        uint32_t m = (uint32_t)kExpBitsMax;
        for (int j = 15; j > kExpBitsMax; --j) open += need_mass[j];
        while (m > (uint32_t)kExpBitsMin && open + need_mass[m] <= 6e-5f) {
            open += need_mass[m];
            --m;
        }
        aux.expm = m;
    }
    __syncthreads();
    const float d = (float)(tid - T.zero_point);
    aux.val[tid] = T.raw_symbols ? (uint16_t)tid : __half_as_ushort(__float2half_rn(__fmul_rn(T.scale, d)));
    __syncthreads();
    {
        uint32_t used = aux.offset[ENTRO_MAX_CODE_LEN] + count[ENTRO_MAX_CODE_LEN];
        if ((uint32_t)tid >= used) aux.sorted[tid] = 0;   // never indexed; keep it defined
    }
    __syncthreads();

    if (aux.oct) {
        const uint32_t entries = 1u << lut_bits;
        for (uint32_t i = first; i < entries; i += stride) {
            uint32_t window = i << (32 - lut_bits);
            uint32_t used = 0;
            uint32_t v[8];
            bool ok = true;
            for (int k = 0; k < 8; ++k) {
                uint32_t sl;
                uint32_t sym = range_decode(aux, window, (uint32_t)lut_bits - used, sl);
                if (sl == 0) {
                    ok = false;
                    break;
                }
                v[k] = aux.val[sym];
                used += sl;
                window <<= sl;   // sl <= lut_bits < 32
            }
            uint4 e = make_uint4(0u, 0u, 0u, 0u);
            if (ok) e = make_uint4(v[0] | (v[1] << 16), v[2] | (v[3] << 16), v[4] | (v[5] << 16), v[6] | (v[7] << 16));
            out.oct_val[i] = e;
            out.oct_len[i] = ok ? (uint8_t)used : (uint8_t)0;
        }
    }
    {
        // cell (e5, mant): windows that start with r ones and a zero, followed by the bits ~mant
        const uint32_t kExpBits = aux.expm;
        for (uint32_t i = first; i < (32u << kExpBits); i += stride) {
            const uint32_t e5 = i >> kExpBits, mant = i & ((1u << kExpBits) - 1u);
            const uint32_t r = (30u - e5) & 31u;
            const uint32_t avail = 31u - r;                               // window bits after the zero
            const uint32_t mb = avail < kExpBits ? avail : kExpBits;
            uint32_t entry = kEscLen;
            if ((mant & ((1u << (kExpBits - mb)) - 1u)) == 0u) {          // else no window maps here
                const uint32_t mt = mant >> (kExpBits - mb);
                const uint32_t vb = ~mt & ((1u << mb) - 1u);
                const uint32_t ones = r ? (0xffffffffu << (32u - r)) : 0u;
                const uint32_t v_lo = ones | (vb << (avail - mb));
                uint32_t sl;
                uint32_t sym = range_decode(aux, v_lo, aux.max_len, sl);
                bool ok = sl != 0 && sl <= r + 1u + mb;
                if (ok && i == 0) {
                    // the window of 32 ones converts to 0.0f and lands in this cell as well
                    uint32_t sl1;
                    uint32_t sym1 = range_decode(aux, 0xffffffffu, aux.max_len, sl1);
                    ok = sl1 == sl && sym1 == sym;
                }
                if (ok) entry = ((uint32_t)aux.val[sym] << 16) | sl;
            }
            (aux.oct ? out.exp_small : out.exp_lut())[i] = entry;
        }
    }
    const uint32_t* src = reinterpret_cast<const uint32_t*>(&aux);
    uint32_t* dst = reinterpret_cast<uint32_t*>(&out.aux);
    if (blockIdx.y == 0)
        for (uint32_t i = tid; i < sizeof(DecodeAux) / 4; i += 256) dst[i] = src[i];
}

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
__device__ __forceinline__ LutKey lut_key(uint32_t expm, uint32_t lane)
{
    LutKey k;
    k.mask = ((32u << expm) - 1u) << (11u - expm);
    k.lane = (lane & ((32u >> (expm - 4u)) - 1u)) * 4u;
    return k;
}

// Cell of the exponent-indexed table for an inverted window, in this lane's copy.
__device__ __forceinline__ uint32_t exp_lookup(LutKey key, uint32_t inv_window)
{
    const uint32_t fb = __float_as_uint(__uint2float_rz(inv_window));
    const uint32_t a = ((fb >> 12) & key.mask) | key.lane;
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

// Reader of the grouped lookups of 8-bit alphabets: two consecutive stream words
// (complemented) in registers and a bit position whose low five bits say where in w0 the
// next code starts.  Only those five bits and bit 5 (has a word boundary been crossed?) are
// ever used, so the upper bits of pos may hold anything.
struct Cur {
    uint32_t w0, w1;
    uint32_t pos;
    uint32_t next;            // shared-window address of the word after w1
};

__device__ __forceinline__ void cur_init(Cur& c, uint32_t bit_addr)
{
    const uint32_t a = (bit_addr >> 5) << 2;
    c.w0 = ~lds32(a);
    c.w1 = ~lds32(a + 4);
    c.next = a + 8;
    c.pos = bit_addr;
}

// Shared-window bit address the reader stands at.
__device__ __forceinline__ uint32_t cur_bit_addr(const Cur& c) { return (c.next - 8u) * 8u + (c.pos & 31u); }

// One group of lookups, hand-scheduled.  The group sees the 32 bits that start at the
// reader's position (one funnel shift of the two words) and nothing behind them: a lookup
// reads them shifted left by the lengths found before it (a funnel shift uses the low five
// bits of its count), zeros moving in from the right.  Those
// zeros cannot mislead a lookup whose code ends inside the 32 bits: a cell is resolved only
// if every window that maps to it begins with the same code, whatever follows.  s is the sum
// of the G entries: the group stands iff (s & 0xffe0) == 0, that is, every cell was resolved
// (an unresolved one adds 64) and fewer than 32 bits were used, so all codes did end inside
// the 32 bits.  Then the position moves on by s and, if that crosses into the next word
// (bit 5 of the position flips), w1 becomes w0 and one new word is pulled in, predicated.
// If the group does not stand the caller repairs it from rewind_group, which needs only
// pos, next and s.
#define ENTRO_LOOKUP(dst, win)                       \
    "cvt.rz.f32.u32 f, " win ";\n\t"                  \
    "mov.b32 a, f;\n\t"                               \
    "shr.u32 a, a, 12;\n\t"                           \
    "lop3.b32 a, a, %8, %7, 0xEA;\n\t"                \
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
    "@p ld.shared.b32 t, [%3];\n\t"                   \
    "@p add.u32 %3, %3, 4;\n\t"                       \
    "@p not.b32 %1, t;\n\t"

__device__ __forceinline__ void group4(Cur& c, LutKey key, uint32_t& pk0, uint32_t& pk1, uint32_t& s)
{
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
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
        : "+r"(c.w0), "+r"(c.w1), "+r"(c.pos), "+r"(c.next), "=&r"(pk0), "=&r"(pk1), "=&r"(s)
        : "r"(key.lane), "r"(key.mask));
}

__device__ __forceinline__ void group2(Cur& c, LutKey key, uint32_t& pk0, uint32_t& s)
{
    __attribute__((unused)) uint32_t unused;   // operand slot of the second pair, which a group of two does not have
    asm volatile(
        "{\n\t"
        ".reg .pred p;\n\t"
        ".reg .b32 t, w, a, h, e0, e1;\n\t"
        ".reg .f32 f;\n\t" ENTRO_OPEN ENTRO_LOOKUP("e0", "h")
        "shf.l.wrap.b32 w, 0, h, e0;\n\t" ENTRO_LOOKUP("e1", "w")
        "add.u32 %6, e0, e1;\n\t"
        "prmt.b32 %4, e0, e1, 0x7632;\n\t"
        "mov.b32 %5, 0;\n\t" ENTRO_MOVE_ON "}"
        : "+r"(c.w0), "+r"(c.w1), "+r"(c.pos), "+r"(c.next), "=&r"(pk0), "=&r"(unused), "=&r"(s)
        : "r"(key.lane), "r"(key.mask));
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
            ".reg .pred p;\n\t"
            ".reg .b32 t, w, a, h, e0, e1;\n\t"
            ".reg .f32 f;\n\t" ENTRO_OPEN ENTRO_LOOKUP("e0", "h")
            "shf.l.wrap.b32 w, 0, h, e0;\n\t" ENTRO_LOOKUP("e1", "w")
            "shf.l.wrap.b32 w, 0, w, e1;\n\t" ENTRO_LOOKUP("%5", "w")
            "add.u32 %6, e0, e1;\n\t"
            "add.u32 %6, %6, %5;\n\t"
            "prmt.b32 %4, e0, e1, 0x7632;\n\t" ENTRO_MOVE_ON "}"
            : "+r"(c.w0), "+r"(c.w1), "+r"(c.pos), "+r"(c.next), "=&r"(first), "=&r"(second), "=&r"(s)
            : "r"(key.lane), "r"(key.mask));
    else
        asm volatile(
            "{\n\t"
            ".reg .pred p;\n\t"
            ".reg .b32 t, w, a, h, e1, e2;\n\t"
            ".reg .f32 f;\n\t" ENTRO_OPEN ENTRO_LOOKUP("%4", "h")
            "shf.l.wrap.b32 w, 0, h, %4;\n\t" ENTRO_LOOKUP("e1", "w")
            "shf.l.wrap.b32 w, 0, w, e1;\n\t" ENTRO_LOOKUP("e2", "w")
            "add.u32 %6, %4, e1;\n\t"
            "add.u32 %6, %6, e2;\n\t"
            "prmt.b32 %5, e1, e2, 0x7632;\n\t" ENTRO_MOVE_ON "}"
            : "+r"(c.w0), "+r"(c.w1), "+r"(c.pos), "+r"(c.next), "=&r"(first), "=&r"(second), "=&r"(s)
            : "r"(key.lane), "r"(key.mask));
}
#undef ENTRO_LOOKUP
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
    return (c.next - 8u - 4u * crossed) * 8u + (before & 31u);
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

// Chunk whose bytes have been asked for.  meta packs what the staging needs: ring offset /
// 16 (12 bits), bytes / 16 (12 bits), ticket modulo 4 (2 bits), kind (2 bits), copy issued
// (1 bit).  Everything else is re-read from the chunk's index slot when it is decoded.
struct Ready {
    uint32_t c;                // or kNone
    uint32_t meta;
    __device__ __forceinline__ uint32_t at() const { return (meta & 0xfffu) << 4; }
    __device__ __forceinline__ uint32_t bytes() const { return ((meta >> 12) & 0xfffu) << 4; }
    __device__ __forceinline__ uint32_t ticket() const { return (meta >> 24) & 3u; }
    __device__ __forceinline__ uint32_t kind() const { return (meta >> 26) & 3u; }
    __device__ __forceinline__ bool issued() const { return (meta >> 28) & 1u; }
};
__device__ __forceinline__ uint32_t ready_meta(uint32_t at, uint32_t bytes, uint32_t ticket, uint32_t kind)
{
    return (at >> 4) | ((bytes >> 4) << 12) | ((ticket & 3u) << 24) | (kind << 26);
}

__device__ __forceinline__ unsigned long long lds64(uint32_t addr)
{
    unsigned long long v;
    asm volatile("ld.shared.b64 %0, [%1];" : "=l"(v) : "r"(addr));
    return v;
}

// Ask for chunk c's index entries to be copied into the slot at shared address `slot`
// (lanes 0..15 two sub-block lengths each, lanes 16 and 17 one offset each).  Nothing is
// held in registers while the copies are in flight.
__device__ __forceinline__ void fetch_index(const DevTensor& T, uint32_t c, uint32_t slot, uint32_t lane)
{
    if (c != kNone) {
        if (lane < 16u) {
            const char* src = reinterpret_cast<const char*>(T.sub_len + (uint64_t)c * kSubBlocks) + lane * 4u;
            asm volatile("cp.async.ca.shared.global [%0], [%1], 4;" ::"r"(slot + lane * 4u), "l"(src) : "memory");
        } else if (lane < 18u) {
            const uint64_t* src = T.offsets + c + (lane - 16u);
            asm volatile("cp.async.ca.shared.global [%0], [%1], 8;" ::"r"(slot + 64u + (lane - 16u) * 8u), "l"(src)
                         : "memory");
        }
    }
    asm volatile("cp.async.commit_group;" ::: "memory");
}

__device__ __forceinline__ void issue_copy(const WarpCtx& cx, const DevTensor& T, Ready& r, uint64_t byte0, uint32_t lane)
{
    if (lane == 0)
        bulk_load(cx.stage_addr + r.at(), reinterpret_cast<const char*>(T.stream) + byte0, r.bytes(),
                  cx.bar + 8u * (r.ticket() & 1u));
    r.meta |= 1u << 28;
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
__device__ __forceinline__ Ready prepare(WarpCtx& cx, const DevTensor& T, uint32_t stage_bytes, uint32_t* status,
                                         uint32_t c, uint32_t slot, const Ready& prev, uint32_t lane)
{
    Ready r;
    r.c = c;
    r.meta = ready_meta(0, 0, 0, kSkip);
    asm volatile("cp.async.wait_all;" ::: "memory");
    __syncwarp();
    if (c == kNone) return r;
    const uint64_t off0 = lds64(slot + 64u), off1 = lds64(slot + 72u);
    uint64_t byte0, byte1;
    chunk_bytes(off0, off1, byte0, byte1);
    if (off1 < off0 || off1 - off0 > 32ull * 65535ull || byte1 > T.stream_words * 4) {
        if (lane == 0) atomicOr(status, kStatCorrupt);
        return r;
    }
    const uint32_t sub = T.chunk_symbols / kSubBlocks;
    const bool full = (uint64_t)(c + 1) * T.chunk_symbols <= T.n;
    const uint32_t bytes = (uint32_t)(byte1 - byte0);
    if (!full || (sub & 7u) || bytes > stage_bytes || cx.dead()) {
        r.meta = ready_meta(0, 0, 0, kGeneral);
        return r;
    }
    // ring placement: behind the previous chunk's bytes, else at the start if that does not
    // overlap them, else at the start once the previous chunk has been decoded
    uint32_t at = 0;
    bool now = true;
    if (prev.c != kNone && prev.kind() == kStaged) {
        const uint32_t end = prev.at() + prev.bytes();
        if (end + bytes <= stage_bytes) at = end;
        else if (bytes > prev.at()) now = false;
    }
    r.meta = ready_meta(at, bytes, cx.state, kStaged);
    cx.state++;
    if (now) issue_copy(cx, T, r, byte0, lane);
    else if (lane == 0)   // no room yet: at least bring the bytes into L2 while the previous chunk is decoded
        asm volatile("cp.async.bulk.prefetch.L2.global [%0], %1;" ::"l"(reinterpret_cast<const char*>(T.stream) + byte0),
                     "r"(bytes)
                     : "memory");
    return r;
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
            if (!oct) e = exp_lookup(lut_key(aux->expm, lane), ~r.hi);
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
            } else {
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
}

// ------------------------------------------------------------------ what happens to decoded values

__device__ __forceinline__ uint4 lds128(uint32_t addr)
{
    uint4 v;
    asm volatile("ld.shared.v4.b32 {%0,%1,%2,%3}, [%4];" : "=r"(v.x), "=r"(v.y), "=r"(v.z), "=r"(v.w) : "r"(addr));
    return v;
}

// Plain decode: the 8 values of this lane's next group go to the output tensor.  A lane's
// consecutive groups are 32 groups apart, so one call per lane writes 512 contiguous bytes.
struct EmitStore {
    uint4* dst;
    __device__ __forceinline__ void operator()(uint4 v)
    {
        __stcs(dst, v);
        dst += kSubBlocks;
    }
    __device__ __forceinline__ void finish() {}
};

// Integer output (the form the paper's decoder produces): the tables hold the symbols
// themselves in their 16-bit value fields; a group of 8 leaves as 8 bytes ...
struct EmitBytes {
    uint2* dst;
    __device__ __forceinline__ void operator()(uint4 v)
    {
        __stcs(dst, make_uint2(__byte_perm(v.x, v.y, 0x6420), __byte_perm(v.z, v.w, 0x6420)));
        dst += kSubBlocks;
    }
};

// ... or, for 4-bit symbols, as 4 bytes of two nibbles each, the earlier symbol low.
struct EmitNibbles {
    uint32_t* dst;
    __device__ __forceinline__ void operator()(uint4 v)
    {
        const uint32_t a = __byte_perm(v.x, v.y, 0x6420), b = __byte_perm(v.z, v.w, 0x6420);   // s0..s3, s4..s7
        const uint32_t ta = a | (a >> 4), tb = b | (b >> 4);                                   // bytes 0 and 2 hold the pairs
        __stcs(dst, __byte_perm(ta, tb, 0x6420));
        dst += kSubBlocks;
    }
};

// Fused matrix-vector product: the 8 values are weights of one row of W (stored [rows, cols],
// cols a multiple of 256, so the 32 lanes of a step stay inside one row) and meet the 8
// matching entries of x of every token, staged in shared memory as fp16 token after token
// (tokens beyond the batch are zeros); products and sums in fp32, one accumulator per token.
// When the row ends the warp adds its lanes up and adds the results to the row's fp32
// accumulators.
template <int B>
struct EmitDot {
    uint32_t xaddr;       // shared-window address of x[0][col .. col + 8) for this lane's next group
    uint32_t xlane;       // the same at the start of a row
    uint32_t xstride;     // bytes from one token's x to the next
    uint32_t left;        // steps left in the current row
    uint32_t rs;          // steps per row (cols / 256)
    float acc[B];
    float* yrow;          // fp32 accumulator of the current row, first token
    uint32_t rows, batch;
    uint32_t lane;

    __device__ __forceinline__ void flush()
    {
#pragma unroll
        for (int b = 0; b < B; ++b) {
            float v = acc[b];
#pragma unroll
            for (int d = 16; d > 0; d >>= 1) v += __shfl_xor_sync(0xffffffffu, v, d);
            if (lane == 0 && (uint32_t)b < batch) atomicAdd(yrow + (uint64_t)b * rows, v);
            acc[b] = 0.f;
        }
        ++yrow;
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
        if (--left == 0u) flush();
    }
    __device__ __forceinline__ void finish()
    {
        if (left != rs) flush();     // the chunk ended inside a row
    }
};

// 8-bit alphabets, eight symbols per turn.  G = 2, 3 (as 3 + 3 + 2), 4: groups of that many
// lookups, each checked.  G = 8: two groups of four under one check, for streams whose groups
// of four almost never fail; if either failed, both are done again one by one.
template <int K, int G, class Emit>
__device__ __forceinline__ uint32_t rows_single(uint32_t start, uint32_t* status, LutKey key, Emit& emit, uint32_t sub)
{
    Cur r;
    cur_init(r, start);
    for (uint32_t t0 = 0; t0 < sub; t0 += 8) {
        uint32_t pk[4];
        bool again = G == 4;
        if (G == 8) {
            uint32_t s0, s1;
            group4(r, key, pk[0], pk[1], s0);
            group4(r, key, pk[2], pk[3], s1);
            if (__builtin_expect(((s0 | s1) & 0xffe0u) != 0u, 0)) {
                // back over both: the position moved by s0 + s1, the words by one per flip of bit 5
                const uint32_t p1 = r.pos - s1, p0 = p1 - s0;
                const uint32_t steps = (((p0 ^ p1) >> 5) & 1u) + (((p1 ^ r.pos) >> 5) & 1u);
                cur_init(r, (r.next - 8u - 4u * steps) * 8u + (p0 & 31u));
                again = true;
            }
        }
        if (G == 4 || G == 8) {
            if (again) {
#pragma unroll
                for (int g = 0; g < 2; ++g) {
                    uint32_t s;
                    group4(r, key, pk[2 * g], pk[2 * g + 1], s);
                    if (__builtin_expect((s & 0xffe0u) != 0u, 0)) repair_quad<K>(r, status, key, s, pk[2 * g], pk[2 * g + 1]);
                }
            }
        } else if (G == 3) {
            uint32_t s, a2, b0;
            group3<false>(r, key, pk[0], a2, s);
            if (__builtin_expect((s & 0xffe0u) != 0u, 0)) repair_triple<K, false>(r, status, key, s, pk[0], a2);
            group3<true>(r, key, b0, pk[2], s);
            if (__builtin_expect((s & 0xffe0u) != 0u, 0)) repair_triple<K, true>(r, status, key, s, b0, pk[2]);
            pk[1] = __byte_perm(a2, b0, 0x7632);
            group2(r, key, pk[3], s);
            if (__builtin_expect((s & 0xffe0u) != 0u, 0)) repair_pair<K>(r, status, key, s, pk[3]);
        } else {
#pragma unroll
            for (int g = 0; g < 4; ++g) {
                uint32_t s;
                group2(r, key, pk[g], s);
                if (__builtin_expect((s & 0xffe0u) != 0u, 0)) repair_pair<K>(r, status, key, s, pk[g]);
            }
        }
        emit(make_uint4(pk[0], pk[1], pk[2], pk[3]));
    }
    return cur_bit_addr(r);
}

// 4-bit alphabets: eight symbols per lookup.
template <int K, class Emit>
__device__ __forceinline__ uint32_t rows_oct(uint32_t start, uint32_t* status, Emit& emit, uint32_t sub)
{
    Win r;
    win_init<false>(r, (start >> 5) << 2, start & 31u);
    for (uint32_t t0 = 0; t0 < sub; t0 += 8) {
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
__device__ __forceinline__ uint32_t rows_any(const DecodeAux* aux, uint32_t start, uint32_t* status, Emit& emit, uint32_t sub,
                                             uint32_t lane)
{
    if (aux->oct) return rows_oct<K>(start, status, emit, sub);
    const LutKey key = lut_key(aux->expm, lane);
    switch (aux->group) {
        case 8u: return rows_single<K, 8>(start, status, key, emit, sub);
        case 4u: return rows_single<K, 4>(start, status, key, emit, sub);
        case 3u: return rows_single<K, 3>(start, status, key, emit, sub);
        default: return rows_single<K, 2>(start, status, key, emit, sub);
    }
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
    uint32_t incl = bits;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        uint32_t t = __shfl_up_sync(0xffffffffu, incl, d);
        if (lane >= (uint32_t)d) incl += t;
    }
    const uint32_t total = __shfl_sync(0xffffffffu, incl, 31);
    const uint64_t off0 = lds64(slot + 64u), off1 = lds64(slot + 72u);
    if (off1 - off0 != (uint64_t)total) {       // the recorded lengths do not add up to the chunk
        if (lane == 0) atomicOr(status, kStatCorrupt);
        L.kind = kSkip;
        return L;
    }
    const uint32_t excl = incl - bits;
    if (L.kind == kGeneral) {
        L.start = excl;
        L.end = bits;
    } else {
        const uint32_t byte0_bits = (uint32_t)off0 & ~127u;    // bit offset of the copied bytes' start, modulo 2^32
        L.start = (cx.stage_addr + r.at()) * 8u + ((uint32_t)off0 - byte0_bits) + excl;
        L.end = L.start + bits;
    }
    return L;
}

template <int K, int kSink>
__device__ __forceinline__ void decode_finish(WarpCtx& cx, uint32_t* status, Ready& r, Lane L, uint32_t lane)
{
    constexpr int kBatch = kGemvBatchOf<kSink>;
    constexpr bool kGemv = kBatch > 0;
    if (L.kind == kSkip) return;
    const DevTensor& T = *tensor_ptr<K>();
    const GemvTensor* G = kGemv ? gemv_ptr<K>() : nullptr;
    if (L.kind == kStaged) {
        if (!r.issued()) issue_copy(cx, T, r, (T.offsets[r.c] >> 3) & ~15ull, lane);
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
    const uint32_t sub = T.chunk_symbols / kSubBlocks;
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
        em.yrow = G->y32 + row0;
        em.rows = G->rows;
        em.batch = G->batch;
        stood = rows_any<K>(aux_ptr<K>(), L.start, status, em, sub, lane);
        em.finish();
    } else if (kSink == kSinkBytes) {
        EmitBytes em;
        em.dst = reinterpret_cast<uint2*>(reinterpret_cast<uint8_t*>(T.out) + (uint64_t)r.c * T.chunk_symbols + lane * 8u);
        stood = rows_any<K>(aux_ptr<K>(), L.start, status, em, sub, lane);
    } else if (kSink == kSinkNibbles) {
        EmitNibbles em;
        em.dst = reinterpret_cast<uint32_t*>(reinterpret_cast<uint8_t*>(T.out) + (((uint64_t)r.c * T.chunk_symbols) >> 1) +
                                             lane * 4u);
        stood = rows_any<K>(aux_ptr<K>(), L.start, status, em, sub, lane);
    } else {
        EmitStore em;
        em.dst = reinterpret_cast<uint4*>(T.out + (uint64_t)r.c * T.chunk_symbols + lane * 8u);
        stood = rows_any<K>(aux_ptr<K>(), L.start, status, em, sub, lane);
        em.finish();
    }
    // the lane must stand exactly at the end of its sub-block
    if (stood != L.end) atomicOr(status, kStatCorrupt);
    __syncwarp();   // all lanes are done with these bytes before the ring reuses them
}

// ------------------------------------------------------------------ persistent kernel

// item_start[t] = first work item of tensor t, item_start[ntensors] = number of items; an
// item is up to tensors[t].item_chunks consecutive chunks of one tensor.
// kSink says where the decoded values go.  With kSinkGemv they are not stored: gemv[t]
// describes the matrix-vector product they enter (the fused decode + dequantise + GEMV of a
// batch-1 token step).
template <int K, int kSink>
__global__ void __launch_bounds__(1024, 1) decode_kernel(const DevTensor* __restrict__ tensors, int ntensors,
                                                         const uint32_t* __restrict__ item_start,
                                                         const TensorTables* __restrict__ tables,
                                                         uint32_t stage_bytes,
                                                         uint32_t* __restrict__ control,
                                                         const GemvTensor* __restrict__ gemv, uint32_t rings_at)
{
    constexpr int kBatch = kGemvBatchOf<kSink>;
    constexpr bool kGemv = kBatch > 0;
    // layout: [tables][aux][tensor]([gemv descriptor][x])[per-warp rings][over-read pad][mbarriers][index slots][item + claim slots]
    if (smem_addr(smem) != kSmemBase) {   // the lookups' address arithmetic would be wrong: refuse to run
        if (threadIdx.x == 0) atomicOr(control + 1, kStatInternal);
        return;
    }
    DecodeAux* s_aux = aux_ptr<K>();
    DevTensor* s_tensor = tensor_ptr<K>();
    const uint32_t warps = blockDim.x >> 5;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t kRings = rings_at;          // rings_offset<K>(kGemv, bytes of staged x)
    const uint32_t after = kRings + warps * stage_bytes + kOverRead;          // offset in smem, a multiple of 16
    const uint32_t slots = after + warps * 16u;
    volatile uint32_t* s_item = reinterpret_cast<volatile uint32_t*>(smem + slots + warps * 2u * kSlotBytes);   // [2]
    uint32_t* s_claim = const_cast<uint32_t*>(s_item) + 2;                                                     // [2]
    uint32_t* status = control + 1;

    WarpCtx cx;
    cx.stage_addr = kSmemBase + kRings + warp * stage_bytes;
    cx.bar = kSmemBase + after + warp * 16u;
    cx.idx_addr = kSmemBase + slots + warp * 2u * kSlotBytes;
    cx.state = 0;

    if (lane == 0) {
        mbar_init(cx.bar, 1);
        mbar_init(cx.bar + 8u, 1);
    }
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
            const uint4* ga = reinterpret_cast<const uint4*>(&tt->aux);
            uint4* sa = reinterpret_cast<uint4*>(s_aux);
            for (uint32_t i = threadIdx.x; i < sizeof(DecodeAux) / 16; i += blockDim.x) sa[i] = __ldg(ga + i);
            const uint4* gt = reinterpret_cast<const uint4*>(tensors + cur);
            uint4* st = reinterpret_cast<uint4*>(s_tensor);
            for (uint32_t i = threadIdx.x; i < sizeof(DevTensor) / 16; i += blockDim.x) st[i] = __ldg(gt + i);
            if (kGemv) {
                const uint4* gg = reinterpret_cast<const uint4*>(gemv + cur);
                uint4* sg = reinterpret_cast<uint4*>(gemv_ptr<K>());
                if (threadIdx.x < sizeof(GemvTensor) / 16) sg[threadIdx.x] = __ldg(gg + threadIdx.x);
                // x of the batch's tokens, then zeros for the accumulators that have no token
                const uint4* gx = reinterpret_cast<const uint4*>(gemv[cur].x);      // cols is a multiple of 256
                uint4* sx = reinterpret_cast<uint4*>(smem + kGemvX<K>);
                const uint32_t n16 = gemv[cur].cols / 8u;
                const uint32_t have = n16 * gemv[cur].batch, want = n16 * (uint32_t)kBatch;
                for (uint32_t i = threadIdx.x; i < want; i += blockDim.x)
                    sx[i] = i < have ? __ldg(gx + i) : make_uint4(0u, 0u, 0u, 0u);
            }
            if (__ldg(&tt->aux.oct)) {
                const uint4* g1 = tt->oct_val;
                uint4* s1 = reinterpret_cast<uint4*>(smem);
                for (uint32_t i = threadIdx.x; i < (1u << K); i += blockDim.x) s1[i] = __ldg(g1 + i);
                const uint4* g2 = reinterpret_cast<const uint4*>(tt->oct_len);
                uint4* s2 = reinterpret_cast<uint4*>(smem + (16u << K));
                for (uint32_t i = threadIdx.x; i < (1u << K) / 16; i += blockDim.x) s2[i] = __ldg(g2 + i);
                uint32_t* s3 = reinterpret_cast<uint32_t*>(smem + (17u << K));
                for (uint32_t i = threadIdx.x; i < (uint32_t)kExpEntriesMin; i += blockDim.x) s3[i] = __ldg(tt->exp_small + i);
            } else {
                // cell-major copies, 64 KB in all: word w holds cell w / copies
                uint32_t* s1 = reinterpret_cast<uint32_t*>(smem);
                const uint32_t shift = 9u - __ldg(&tt->aux.expm);       // log2 of the number of copies
                for (uint32_t w = threadIdx.x; w < (uint32_t)kExpEntriesMax; w += blockDim.x)
                    s1[w] = __ldg(tt->exp_lut() + (w >> shift));
            }
            __syncthreads();
        }
        const DevTensor& T = *s_tensor;
        const uint32_t chunks_per_item = T.item_chunks;
        const uint32_t first = (item - __ldg(item_start + cur)) * chunks_per_item;

        // The warps share out the item's chunks.  Each warp, per turn: start the bulk copy of
        // chunk i + 1 (its offsets arrived a turn ago), work out the lanes' positions in chunk
        // i, ask for the index entries of chunk i + 2 in the slot that frees, decode chunk i.
        auto claim = [&]() -> uint32_t {
            uint32_t k = 0;
            if (lane == 0) k = atomicAdd(&s_claim[slot], 1u);
            k = __shfl_sync(0xffffffffu, k, 0);
            return k < min(chunks_per_item, T.n_chunks - first) ? first + k : kNone;
        };
        Ready r0;
        r0.c = kNone;
        r0.meta = ready_meta(0, 0, 0, kSkip);
        uint32_t sp = cx.idx_addr;                  // slot of the chunk fetched last
        uint32_t c2 = claim();
        fetch_index(T, c2, sp, lane);
        while (true) {
            Ready r1 = prepare(cx, T, stage_bytes, status, c2, sp, r0, lane);
            const uint32_t other = cx.idx_addr + (sp == cx.idx_addr ? kSlotBytes : 0u);
            const Lane L = decode_start<K>(cx, status, r0, other, lane);
            __syncwarp();                           // every lane has read the slot before it is refilled
            c2 = r1.c == kNone ? kNone : claim();
            fetch_index(T, c2, other, lane);
            decode_finish<K, kSink>(cx, status, r0, L, lane);
            if (r1.c == kNone) break;
            r0 = r1;
            sp = other;
        }
        asm volatile("cp.async.wait_all;" ::: "memory");
        __syncthreads();   // tables may be replaced; s_item / s_claim [slot ^ 1] are now visible
        slot ^= 1u;
    }
    // A warp that gave up on a bulk copy lets it land (bounded) before its buffer goes away.
    const uint32_t issued = cx.state & 0x7fffffffu;
    if (cx.dead() && issued) (void)mbar_wait(cx.bar + 8u * ((issued - 1) & 1u), ((issued - 1) >> 1) & 1u);
}

struct Shape {
    size_t smem;
    uint32_t stage_bytes;
};

// Shared memory of one CTA for a launch shape; stage_bytes == 0 if it cannot fit.
Shape shape_for(const DecodeConfig& cfg, int max_smem, bool gemv = false, uint32_t x_bytes = 0)
{
    size_t fixed = lut_bytes(cfg.lut_bits) + sizeof(DecodeAux) + sizeof(DevTensor) + 128 + kOverRead;
    if (gemv) fixed += sizeof(GemvTensor) + x_bytes;
    size_t per_warp_fixed = 16 + 2 * kSlotBytes;   // two mbarriers, two index slots
    size_t tail = 16;
    size_t budget = (size_t)max_smem / cfg.ctas_per_sm;
    if (cfg.ctas_per_sm > 1) budget -= 1024;   // per-CTA reservation of the driver
    Shape s{0, 0};
    if (budget < fixed + tail + cfg.warps_per_cta * (per_warp_fixed + 1024)) return s;
    size_t avail = (budget - fixed - tail) / cfg.warps_per_cta - per_warp_fixed;
    uint32_t stage = (uint32_t)(avail & ~(size_t)127);
    if (stage > 32768u) stage = 32768u;
    s.stage_bytes = stage;
    s.smem = fixed + tail + cfg.warps_per_cta * (per_warp_fixed + stage);
    return s;
}

template <int K, int kSink>
entro_status launch_decode(Workspace* ws, const DecodeConfig& cfg, const DevTensor* tensors, int ntensors,
                           const uint32_t* item_start, uint32_t total_items, const TensorTables* tables,
                           const GemvTensor* gemv, cudaStream_t s, uint32_t x_bytes)
{
    constexpr bool kGemv = kGemvBatchOf<kSink> > 0;
    Shape sh = shape_for(cfg, ws->max_smem_optin, kGemv, x_bytes);
    if (sh.stage_bytes == 0) return ENTRO_ERR_UNSUPPORTED;
    static int configured_smem[64] = {0};      // per instantiation of this template
    if ((int)sh.smem > configured_smem[ws->device]) {
        ENTRO_CUDA(cudaFuncSetAttribute(decode_kernel<K, kSink>, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                        (int)sh.smem));
        configured_smem[ws->device] = (int)sh.smem;
    }
    uint32_t grid = (uint32_t)ws->sm_count * cfg.ctas_per_sm;
    if (grid > total_items) grid = total_items;
    const bool timed = ws->prof_used < ws->prof_cap;
    if (timed) ENTRO_CUDA(cudaEventRecord(ws->prof_start[ws->prof_used], s));
    decode_kernel<K, kSink><<<grid, cfg.warps_per_cta * 32, sh.smem, s>>>(
        tensors, ntensors, item_start, tables, sh.stage_bytes, ws->control, gemv, rings_offset<K>(kGemv, x_bytes));
    count_launch();
    ENTRO_CUDA(cudaGetLastError());
    if (timed) ENTRO_CUDA(cudaEventRecord(ws->prof_stop[ws->prof_used++], s));
    return ENTRO_OK;
}

template <int kSink>
entro_status launch_decode_sink(Workspace* ws, const DecodeConfig& cfg, const DevTensor* tensors, int ntensors,
                                const uint32_t* item_start, uint32_t total_items, const TensorTables* tables,
                                const GemvTensor* gemv, cudaStream_t s, uint32_t x_bytes = 0)
{
    switch (cfg.lut_bits) {
        case 10: return launch_decode<10, kSink>(ws, cfg, tensors, ntensors, item_start, total_items, tables, gemv, s, x_bytes);
        case 11: return launch_decode<11, kSink>(ws, cfg, tensors, ntensors, item_start, total_items, tables, gemv, s, x_bytes);
        case 12: return launch_decode<12, kSink>(ws, cfg, tensors, ntensors, item_start, total_items, tables, gemv, s, x_bytes);
    }
    return ENTRO_ERR_UNSUPPORTED;
}

// gemv != nullptr: the fused matrix-vector kernel with `batch` accumulators per lane (1, 2,
// 4 or 8) and x_bytes of shared memory for x.
entro_status launch_decode_any(Workspace* ws, const DecodeConfig& cfg, const DevTensor* tensors, int ntensors,
                               const uint32_t* item_start, uint32_t total_items, const TensorTables* tables,
                               cudaStream_t s, const GemvTensor* gemv = nullptr, int sink = kSinkFp16, int batch = 1,
                               uint32_t x_bytes = 0)
{
    if (gemv) {
        switch (batch) {
            case 1: return launch_decode_sink<kSinkGemv>(ws, cfg, tensors, ntensors, item_start, total_items, tables, gemv, s, x_bytes);
            case 2: return launch_decode_sink<kSinkGemv2>(ws, cfg, tensors, ntensors, item_start, total_items, tables, gemv, s, x_bytes);
            case 4: return launch_decode_sink<kSinkGemv4>(ws, cfg, tensors, ntensors, item_start, total_items, tables, gemv, s, x_bytes);
            case 8: return launch_decode_sink<kSinkGemv8>(ws, cfg, tensors, ntensors, item_start, total_items, tables, gemv, s, x_bytes);
        }
        return ENTRO_ERR_UNSUPPORTED;
    }
    switch (sink) {
        case kSinkFp16: return launch_decode_sink<kSinkFp16>(ws, cfg, tensors, ntensors, item_start, total_items, tables, nullptr, s);
        case kSinkBytes: return launch_decode_sink<kSinkBytes>(ws, cfg, tensors, ntensors, item_start, total_items, tables, nullptr, s);
        case kSinkNibbles: return launch_decode_sink<kSinkNibbles>(ws, cfg, tensors, ntensors, item_start, total_items, tables, nullptr, s);
    }
    return ENTRO_ERR_UNSUPPORTED;
}

entro_status validate_desc(const entro_tensor_desc& d, bool need_out = true)
{
    if (d.n == 0) return ENTRO_OK;
    if (!d.stream_dev || !d.index_dev || (need_out && !d.out_fp16_dev)) return ENTRO_ERR_INVALID_ARG;
    if (!aligned(d.stream_dev, 16) || !aligned(d.index_dev, 8) || (need_out && !aligned(d.out_fp16_dev, 16)))
        return ENTRO_ERR_INVALID_ARG;
    if (d.chunk_symbols < kSubBlocks || d.chunk_symbols % kSubBlocks || d.chunk_symbols > ENTRO_MAX_CHUNK_SYMBOLS)
        return ENTRO_ERR_INVALID_ARG;
    if (!codebook_lengths_valid(&d.cb)) return ENTRO_ERR_INVALID_ARG;
    if (num_chunks(d.n, d.chunk_symbols) > 0x7fffffffull) return ENTRO_ERR_UNSUPPORTED;
    if (d.stream_words < ENTRO_STREAM_SLACK_WORDS + 1) return ENTRO_ERR_INVALID_ARG;
    return ENTRO_OK;
}

// How a launch's chunks are cut into work items.  Large items keep the per-item costs (a
// CTA-wide barrier, table reload, pipeline refill) small; the items at the end of the list
// are an eighth of that size so that the CTAs finish together; and a launch with few chunks
// (one layer, one tensor) gets items small enough that every CTA still has several.
struct ItemPlan {
    uint64_t total = 0;        // chunks in the launch
    uint64_t seen = 0;         // chunks of the tensors planned so far
    uint32_t base = 0, tail = 0;
    bool graded = false;
};

ItemPlan plan_items(const DecodeConfig& cfg, const entro_tensor_desc* descs, int ntensors, int sm_count)
{
    ItemPlan p;
    int live = 0;
    for (int i = 0; i < ntensors; ++i)
        if (descs[i].n) {
            p.total += num_chunks(descs[i].n, descs[i].chunk_symbols);
            ++live;
        }
    const uint64_t ctas = (uint64_t)sm_count * cfg.ctas_per_sm;
    uint64_t want = (p.total + ctas * 4 - 1) / (ctas * 4);
    want = (want + cfg.warps_per_cta - 1) / cfg.warps_per_cta * cfg.warps_per_cta;
    if (want < (uint64_t)cfg.warps_per_cta) want = cfg.warps_per_cta;
    p.base = want < (uint64_t)cfg.chunks_per_item ? (uint32_t)want : (uint32_t)cfg.chunks_per_item;
    p.tail = p.base / 8 < (uint32_t)cfg.warps_per_cta ? (uint32_t)cfg.warps_per_cta : p.base / 8;
    p.graded = live >= 8 && p.base >= 8u * (uint32_t)cfg.warps_per_cta;   // a tail item still gives every warp a chunk
    return p;
}

// Device-side form of a descriptor; returns the tensor's number of work items.
uint64_t fill_dev_tensor(const entro_tensor_desc& d, ItemPlan& plan, DevTensor& t)
{
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
    // the last 12 % of the launch's chunks go out in small items; sizes are meant for
    // 4096-symbol chunks and scale down for larger ones, so that an item is as much work
    uint32_t per_item = (plan.graded && (plan.seen + nc) * 100 > plan.total * 88) ? plan.tail : plan.base;
    if (d.chunk_symbols > 4096u) per_item = (uint32_t)((uint64_t)per_item * 4096u / d.chunk_symbols);
    if (per_item < 32u) per_item = 32u;
    t.item_chunks = per_item;
    plan.seen += nc;
    t.raw_symbols = 0;
    t.pad = 0;
    for (int j = 0; j < ENTRO_MAX_SYMBOLS; ++j) t.len[j] = j < d.cb.nsym ? d.cb.len[j] : 0;
    return (nc + t.item_chunks - 1) / t.item_chunks;
}

}  // namespace

// Upload descriptors, build the tables and run the persistent decode kernel.
entro_status decode_batched_locked(Workspace* ws, const entro_tensor_desc* descs, int ntensors, cudaStream_t s,
                                   int sink = kSinkFp16)
{
    const DecodeConfig cfg = decode_config();
    ItemPlan plan = plan_items(cfg, descs, ntensors, ws->sm_count);
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
    int k = 0;
    for (int i = 0; i < ntensors; ++i) {
        if (!descs[i].n) continue;
        hitems[k] = (uint32_t)items;
        items += fill_dev_tensor(descs[i], plan, ht[k]);
        ht[k].raw_symbols = sink == kSinkFp16 ? 0u : 1u;
        if (items > 0x7fffffffull) return ENTRO_ERR_UNSUPPORTED;
        ++k;
    }
    hitems[live] = (uint32_t)items;

    char* base = static_cast<char*>(ws->dev);
    DevTensor* dt = reinterpret_cast<DevTensor*>(base);
    uint32_t* ditems = reinterpret_cast<uint32_t*>(base + tensors_bytes);
    TensorTables* dtables = reinterpret_cast<TensorTables*>(base + upload_bytes);
    ENTRO_CUDA(cudaMemcpyAsync(dt, ht, upload_bytes, cudaMemcpyHostToDevice, s));
    mark_pinned_in_use(ws, s);
    build_tables_kernel<<<dim3((unsigned)live, kTableSlices), 256, 0, s>>>(dt, cfg.lut_bits, dtables, ws->control, nullptr);
    count_launch();
    ENTRO_CUDA(cudaGetLastError());
    return launch_decode_any(ws, cfg, dt, live, ditems, (uint32_t)items, dtables, s, nullptr, sink);
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

extern "C" entro_status entro_decode_symbols_batched(const entro_tensor_desc* descs_host, int ntensors, int packed,
                                                     void* cuda_stream)
{
    if (ntensors < 0 || (ntensors > 0 && !descs_host) || (packed != 0 && packed != 1)) return ENTRO_ERR_INVALID_ARG;
    if (ntensors == 0) return ENTRO_OK;
    for (int i = 0; i < ntensors; ++i) {
        entro_status st = validate_desc(descs_host[i]);
        if (st != ENTRO_OK) return st;
        if (packed && descs_host[i].n && (descs_host[i].cb.nsym > 16 || (descs_host[i].chunk_symbols & 1u)))
            return ENTRO_ERR_INVALID_ARG;
    }
    Guard g;
    Workspace* ws = workspace();
    if (!ws) return ENTRO_ERR_CUDA;
    return decode_batched_locked(ws, descs_host, ntensors, (cudaStream_t)cuda_stream, packed ? kSinkNibbles : kSinkBytes);
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

namespace entro {
namespace {

bool copy_streams_ready(Workspace* ws)
{
    if (ws->copy_in) return true;
    if (cudaStreamCreateWithFlags(&ws->copy_in, cudaStreamNonBlocking) != cudaSuccess) return false;
    if (cudaStreamCreateWithFlags(&ws->copy_out, cudaStreamNonBlocking) != cudaSuccess) return false;
    if (cudaEventCreateWithFlags(&ws->ev_edge, cudaEventDisableTiming) != cudaSuccess) return false;
    for (int i = 0; i < Workspace::kCopyGroups; ++i) {
        if (cudaEventCreateWithFlags(&ws->ev_in[i], cudaEventDisableTiming) != cudaSuccess) return false;
        if (cudaEventCreateWithFlags(&ws->ev_dec[i], cudaEventDisableTiming) != cudaSuccess) return false;
    }
    return true;
}

}  // namespace
}  // namespace entro

// The tensors are cut into groups; uploads, decodes and downloads of different groups
// overlap: group g's streams travel host-to-device on one copy stream while group g - 1 is
// decoded on the caller's stream and group g - 2's fp16 result travels back on another.
extern "C" entro_status entro_decode_dequant_batched_host(const entro_tensor_desc* descs, const entro_host_io* io,
                                                          int ntensors, void* cuda_stream)
{
    if (ntensors < 0 || (ntensors > 0 && (!descs || !io))) return ENTRO_ERR_INVALID_ARG;
    if (ntensors == 0) return ENTRO_OK;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    uint64_t out_bytes = 0;
    for (int i = 0; i < ntensors; ++i) {
        if (!descs[i].n) continue;
        if (!io[i].stream_host || !io[i].index_host || !io[i].out_fp16_host) return ENTRO_ERR_INVALID_ARG;
        entro_status st = validate_desc(descs[i]);
        if (st != ENTRO_OK) return st;
        out_bytes += descs[i].n * 2;
    }
    Guard g;
    Workspace* ws = workspace();
    if (!ws || !copy_streams_ready(ws)) return ENTRO_ERR_CUDA;
    // groups of consecutive tensors, about equal in output bytes
    const uint64_t per_group = out_bytes / Workspace::kCopyGroups + 1;
    // the copy streams start after what the caller has queued, and the caller's stream ends after them
    ENTRO_CUDA(cudaEventRecord(ws->ev_edge, s));
    ENTRO_CUDA(cudaStreamWaitEvent(ws->copy_in, ws->ev_edge, 0));
    ENTRO_CUDA(cudaStreamWaitEvent(ws->copy_out, ws->ev_edge, 0));
    int first = 0, group = 0;
    while (first < ntensors) {
        int last = first;
        uint64_t bytes = 0;
        while (last < ntensors && (bytes < per_group || group == Workspace::kCopyGroups - 1)) bytes += descs[last++].n * 2;
        for (int i = first; i < last; ++i) {
            const entro_tensor_desc& d = descs[i];
            if (!d.n) continue;
            ENTRO_CUDA(cudaMemcpyAsync(const_cast<uint32_t*>(d.stream_dev), io[i].stream_host, d.stream_words * 4,
                                       cudaMemcpyHostToDevice, ws->copy_in));
            ENTRO_CUDA(cudaMemcpyAsync(const_cast<void*>(d.index_dev), io[i].index_host,
                                       entro_index_bytes(d.n, d.chunk_symbols), cudaMemcpyHostToDevice, ws->copy_in));
        }
        ENTRO_CUDA(cudaEventRecord(ws->ev_in[group], ws->copy_in));
        ENTRO_CUDA(cudaStreamWaitEvent(s, ws->ev_in[group], 0));
        entro_status st = decode_batched_locked(ws, descs + first, last - first, s);
        if (st != ENTRO_OK) return st;
        ENTRO_CUDA(cudaEventRecord(ws->ev_dec[group], s));
        ENTRO_CUDA(cudaStreamWaitEvent(ws->copy_out, ws->ev_dec[group], 0));
        for (int i = first; i < last; ++i) {
            const entro_tensor_desc& d = descs[i];
            if (!d.n) continue;
            ENTRO_CUDA(cudaMemcpyAsync(io[i].out_fp16_host, d.out_fp16_dev, d.n * 2, cudaMemcpyDeviceToHost, ws->copy_out));
        }
        first = last;
        ++group;
    }
    ENTRO_CUDA(cudaEventRecord(ws->ev_edge, ws->copy_out));
    ENTRO_CUDA(cudaStreamWaitEvent(s, ws->ev_edge, 0));
    ENTRO_CUDA(cudaStreamSynchronize(s));
    return ENTRO_OK;
}

// ------------------------------------------------------------------ matrix-vector products

namespace entro {
namespace {

// y = fp16(y32) for every tensor of a fused call.
__global__ void __launch_bounds__(256) gemv_finalize_kernel(const GemvTensor* __restrict__ g, int ntensors)
{
    for (int t = blockIdx.y; t < ntensors; t += gridDim.y) {
        const GemvTensor G = g[t];
        const uint32_t n = G.rows * G.batch;      // both are [batch][rows]
        for (uint32_t i = blockIdx.x * blockDim.x + threadIdx.x; i < n; i += gridDim.x * blockDim.x)
            G.y[i] = __half_as_ushort(__float2half_rn(G.y32[i]));
    }
}

// Plain fp16 matrix-vector product (the step that follows an unfused decode): one warp per
// row, 16-byte loads, fp32 products and sums, x read through the read-only path.
__global__ void __launch_bounds__(256) gemv_fp16_kernel(const uint16_t* __restrict__ w, uint32_t rows, uint32_t cols,
                                                        const uint16_t* __restrict__ x, uint16_t* __restrict__ y)
{
    const uint32_t lane = threadIdx.x & 31u;
    const uint32_t warps = (gridDim.x * blockDim.x) >> 5;
    for (uint32_t r = (blockIdx.x * blockDim.x + threadIdx.x) >> 5; r < rows; r += warps) {
        const uint4* wr = reinterpret_cast<const uint4*>(w + (uint64_t)r * cols);
        const uint4* xr = reinterpret_cast<const uint4*>(x);
        float acc = 0.f;
        for (uint32_t i = lane; i < cols / 8u; i += 32u) {
            const uint4 a = __ldcs(wr + i), b = __ldg(xr + i);
            const uint32_t av[4] = {a.x, a.y, a.z, a.w}, bv[4] = {b.x, b.y, b.z, b.w};
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const float2 p = __half22float2(*reinterpret_cast<const __half2*>(&av[k]));
                const float2 q = __half22float2(*reinterpret_cast<const __half2*>(&bv[k]));
                acc = fmaf(p.x, q.x, acc);
                acc = fmaf(p.y, q.y, acc);
            }
        }
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, d);
        if (lane == 0) y[r] = __half_as_ushort(__float2half_rn(acc));
    }
}

}  // namespace
}  // namespace entro

extern "C" entro_status entro_decode_dequant_gemv(const entro_tensor_desc* descs_host, const entro_gemv_io* io_host,
                                                  int ntensors, void* cuda_stream)
{
    if (ntensors < 0 || (ntensors > 0 && (!descs_host || !io_host))) return ENTRO_ERR_INVALID_ARG;
    if (ntensors == 0) return ENTRO_OK;
    uint64_t total_rows = 0;
    uint32_t max_batch = 1;
    for (int i = 0; i < ntensors; ++i) {
        const entro_tensor_desc& d = descs_host[i];
        const entro_gemv_io& g = io_host[i];
        if (d.n == 0) return ENTRO_ERR_INVALID_ARG;
        entro_status st = validate_desc(d, false);
        if (st != ENTRO_OK) return st;
        if (!g.x_fp16_dev || !g.y_fp16_dev || !aligned(g.x_fp16_dev, 16) || !aligned(g.y_fp16_dev, 2))
            return ENTRO_ERR_INVALID_ARG;
        if (g.rows == 0 || g.cols == 0 || (uint64_t)g.rows * g.cols != d.n) return ENTRO_ERR_INVALID_ARG;
        if (g.batch < 1 || g.batch > ENTRO_GEMV_MAX_BATCH || g.reserved != 0) return ENTRO_ERR_INVALID_ARG;
        if ((uint64_t)g.rows * g.batch > 0xffffffffull) return ENTRO_ERR_UNSUPPORTED;
        if (g.cols % 256u || (uint64_t)g.cols * g.batch > kGemvMaxX || d.chunk_symbols % 256u) return ENTRO_ERR_UNSUPPORTED;
        total_rows += (uint64_t)g.rows * g.batch;
        if (g.batch > max_batch) max_batch = g.batch;
    }
    // accumulators per lane: the batch rounded up to 1, 2, 4 or 8; x of that many tokens is staged
    const uint32_t lanes_batch = max_batch <= 1 ? 1u : max_batch <= 2 ? 2u : max_batch <= 4 ? 4u : 8u;
    uint32_t x_bytes = 0;
    for (int i = 0; i < ntensors; ++i) {
        const uint32_t need = (io_host[i].cols * lanes_batch * 2u + 127u) & ~127u;
        if (need > x_bytes) x_bytes = need;
    }
    if (x_bytes > 2u * kGemvMaxX) return ENTRO_ERR_UNSUPPORTED;   // a wide matrix beside a larger batch elsewhere in the call
    cudaStream_t s = (cudaStream_t)cuda_stream;
    Guard guard;
    Workspace* ws = workspace();
    if (!ws) return ENTRO_ERR_CUDA;
    const DecodeConfig cfg = decode_config();
    ItemPlan plan = plan_items(cfg, descs_host, ntensors, ws->sm_count);

    // workspace: [DevTensor x n][item_start][GemvTensor x n] (uploaded) [tables x n][y32]
    const size_t tensors_bytes = (size_t)ntensors * sizeof(DevTensor);
    const size_t items_bytes = (((size_t)ntensors + 1) * 4 + 15) & ~(size_t)15;
    const size_t gemv_bytes = (size_t)ntensors * sizeof(GemvTensor);
    const size_t upload_bytes = tensors_bytes + items_bytes + gemv_bytes;
    const size_t tables_bytes = (size_t)ntensors * sizeof(TensorTables);
    const size_t y32_bytes = (total_rows * 4 + 15) & ~(size_t)15;
    if (!reserve_pinned(ws, upload_bytes)) return ENTRO_ERR_CUDA;
    if (!reserve_device(ws, upload_bytes + tables_bytes + y32_bytes)) return ENTRO_ERR_CUDA;
    char* base = static_cast<char*>(ws->dev);
    char* hbase = static_cast<char*>(ws->pinned);
    DevTensor* ht = reinterpret_cast<DevTensor*>(hbase);
    uint32_t* hitems = reinterpret_cast<uint32_t*>(hbase + tensors_bytes);
    GemvTensor* hg = reinterpret_cast<GemvTensor*>(hbase + tensors_bytes + items_bytes);
    float* y32 = reinterpret_cast<float*>(base + upload_bytes + tables_bytes);
    uint64_t items = 0, row0 = 0;
    for (int i = 0; i < ntensors; ++i) {
        hitems[i] = (uint32_t)items;
        items += fill_dev_tensor(descs_host[i], plan, ht[i]);
        if (items > 0x7fffffffull) return ENTRO_ERR_UNSUPPORTED;
        hg[i].x = static_cast<const uint16_t*>(io_host[i].x_fp16_dev);
        hg[i].y32 = y32 + row0;
        hg[i].y = static_cast<uint16_t*>(io_host[i].y_fp16_dev);
        hg[i].rows = io_host[i].rows;
        hg[i].cols = io_host[i].cols;
        hg[i].batch = io_host[i].batch;
        hg[i].pad[0] = hg[i].pad[1] = hg[i].pad[2] = 0;
        row0 += (uint64_t)io_host[i].rows * io_host[i].batch;
    }
    hitems[ntensors] = (uint32_t)items;
    DevTensor* dt = reinterpret_cast<DevTensor*>(base);
    uint32_t* ditems = reinterpret_cast<uint32_t*>(base + tensors_bytes);
    GemvTensor* dg = reinterpret_cast<GemvTensor*>(base + tensors_bytes + items_bytes);
    TensorTables* dtables = reinterpret_cast<TensorTables*>(base + upload_bytes);
    ENTRO_CUDA(cudaMemcpyAsync(dt, ht, upload_bytes, cudaMemcpyHostToDevice, s));
    mark_pinned_in_use(ws, s);
    build_tables_kernel<<<dim3((unsigned)ntensors, kTableSlices), 256, 0, s>>>(dt, cfg.lut_bits, dtables, ws->control, dg);
    count_launch();
    ENTRO_CUDA(cudaGetLastError());
    entro_status st = launch_decode_any(ws, cfg, dt, ntensors, ditems, (uint32_t)items, dtables, s, dg, kSinkGemv,
                                        (int)lanes_batch, x_bytes);
    if (st != ENTRO_OK) return st;
    dim3 grid(16, (unsigned)(ntensors < 64 ? ntensors : 64));
    gemv_finalize_kernel<<<grid, 256, 0, s>>>(dg, ntensors);
    count_launch();
    ENTRO_CUDA(cudaGetLastError());
    return ENTRO_OK;
}

extern "C" entro_status entro_gemv_fp16(const void* w_fp16_dev, uint32_t rows, uint32_t cols, const void* x_fp16_dev,
                                        void* y_fp16_dev, void* cuda_stream)
{
    if (!w_fp16_dev || !x_fp16_dev || !y_fp16_dev || rows == 0 || cols == 0) return ENTRO_ERR_INVALID_ARG;
    if (cols % 8u || !aligned(w_fp16_dev, 16) || !aligned(x_fp16_dev, 16) || !aligned(y_fp16_dev, 2))
        return ENTRO_ERR_INVALID_ARG;
    int dev = 0, sms = 0;
    ENTRO_CUDA(cudaGetDevice(&dev));
    ENTRO_CUDA(cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev));
    unsigned blocks = (rows + 7u) / 8u;
    const unsigned cap = (unsigned)sms * 8u;
    if (blocks > cap) blocks = cap;
    gemv_fp16_kernel<<<blocks, 256, 0, (cudaStream_t)cuda_stream>>>(
        static_cast<const uint16_t*>(w_fp16_dev), rows, cols, static_cast<const uint16_t*>(x_fp16_dev),
        static_cast<uint16_t*>(y_fp16_dev));
    count_launch();
    ENTRO_CUDA(cudaGetLastError());
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
    ItemPlan plan = plan_items(cfg, descs_host, ntensors, sd->sm_count);

    StaticUpload up;
    uint64_t items = 0;
    int k = 0;
    for (int i = 0; i < ntensors; ++i) {
        if (!descs_host[i].n) continue;
        up.item_start[k] = (uint32_t)items;
        items += fill_dev_tensor(descs_host[i], plan, up.tensors[k]);
        if (items > 0x7fffffffull) return ENTRO_ERR_UNSUPPORTED;
        ++k;
    }
    for (int j = live; j < 16; ++j) up.item_start[j] = (uint32_t)items;
    up.live = live;

    StaticScratch* sc = sd->scratch;
    static_upload_kernel<<<1, 256, 0, s>>>(up, sc);
    count_launch();
    ENTRO_CUDA(cudaGetLastError());
    build_tables_kernel<<<dim3((unsigned)live, kTableSlices), 256, 0, s>>>(sc->tensors, cfg.lut_bits, sc->tables, sc->control, nullptr);
    count_launch();
    ENTRO_CUDA(cudaGetLastError());
    // launch_decode reads only these fields of a workspace; no timing records are taken here
    Workspace ws;
    ENTRO_CUDA(cudaGetDevice(&ws.device));
    ws.sm_count = sd->sm_count;
    ws.max_smem_optin = sd->max_smem_optin;
    ws.control = sc->control;
    st = launch_decode_any(&ws, cfg, sc->tensors, live, sc->item_start, (uint32_t)items, sc->tables, s);
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
    int dev = -1, max_smem = 0;
    if (cudaGetDevice(&dev) == cudaSuccess &&
        cudaDeviceGetAttribute(&max_smem, cudaDevAttrMaxSharedMemoryPerBlockOptin, dev) == cudaSuccess) {
        // the ring of a warp must hold at least 1 KiB
        Shape sh = shape_for(c, max_smem);
        if (sh.stage_bytes < 1024) return ENTRO_ERR_INVALID_ARG;
    }
    decode_config() = c;
    return ENTRO_OK;
}
