// build_tables_kernel: per-tensor decode tables, canonical ranges and the choice of the
// decode mode (Section 3, "Huffman weight encoding": the codes; the table forms are this
// library's).  Included by entro_decode.cu only.
#pragma once

#include "entro_decode_common.cuh"

namespace entro {
namespace {

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
// The grid is (tensors, slices): every block of a tensor works out the small things for
// itself and fills its share of the tables' entries.  Slicing pays when a launch has few
// tensors (one layer: the 4096-entry eight-symbol table took one block 62 us); with a whole
// model in the launch the tensors already fill the GPU and more blocks only repeat the
// small things.
inline unsigned table_slices(int tensors, int sm_count)
{
    const int s = 2 * sm_count / (tensors > 0 ? tensors : 1);
    return (unsigned)(s < 1 ? 1 : s > 8 ? 8 : s);
}
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
    if (gemv) {
        // the fused matrix-vector products: fp32 sums of the rows that span chunks start at zero,
        // and every row is told how many chunks hold a part of it
        const GemvTensor& G = gemv[t];
        const uint32_t n = G.rows * G.batch;
        for (uint32_t i = first; i < n; i += stride) G.y32[i] = 0.f;
        for (uint32_t r = first; r < G.rows; r += stride) {
            const uint64_t a = (uint64_t)r * G.cols, b = a + G.cols - 1u;
            const uint32_t parts = (uint32_t)(b / T.chunk_symbols - a / T.chunk_symbols) + 1u;
            G.pending[r] = parts * 0x10001u;
        }
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
        __shared__ float by_len[33], dist[2][33], fail[9];
        if (tid <= 32) {
            by_len[tid] = tid ? (float)count[tid] * exp2f(-(float)tid) : 0.f;
            dist[0][tid] = tid == 0 ? 1.f : 0.f;
        }
        __syncthreads();
        for (int g = 1; g <= 8; ++g) {
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
            // (with a 4-bit alphabet one symbol is far ahead of the rest and 2^-length says little:
            // there the bit rate alone decides about the eight lookups on one view)
            if (mean_len <= 2.0f && (T.nsym <= 16 || fail[8] < 3e-4f)) aux.group = 16u;
            else if (fail[4] < 3e-4f && mean_len <= 4.0f) aux.group = 8u;   // two groups of four under one check
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
    if (tid == 0) {
        const uint32_t m = aux.expm;
        aux.key_mask = ((32u << m) - 1u) << (11u - m);
        aux.key_lane_mask = (32u >> (m - 4u)) - 1u;
        aux.turns = (T.chunk_symbols % (8u * kSubBlocks)) == 0u ? T.chunk_symbols / (8u * kSubBlocks) : 0u;
        // (9 and 17: groups as in 8 and 16, and the turns per chunk come in pairs; 18: as 16, in fours)
        const bool pairs = aux.turns != 0u && aux.turns % 2u == 0u;
        aux.mode = aux.oct ? 0u : (pairs && (aux.group == 8u || aux.group == 16u)) ? aux.group + 1u : aux.group;
        if (aux.mode == 17u && aux.turns % 4u == 0u) aux.mode = 18u;
    }
    if (tid < 20)
        aux.index_src[tid] = tid < 16 ? reinterpret_cast<unsigned long long>(T.sub_len) + 4ull * tid
                                      : reinterpret_cast<unsigned long long>(T.offsets) + 4ull * (tid - 16);
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

}  // namespace
}  // namespace entro
