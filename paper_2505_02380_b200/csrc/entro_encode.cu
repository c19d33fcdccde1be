// entro_encode: symbols -> bitstream + per-chunk bit-offset index (Section 3: variable
// length codes; segments with known boundaries).  Three passes: bit lengths of every
// sub-block, a prefix sum over chunks, then each sub-block packs its own bits.
// Sub-block l of a chunk is the chunk's 8-symbol groups l, l + 32, l + 64, ... in that
// order (the last group of a chunk may be short).
#include "entro_internal.h"

namespace entro {
namespace {

constexpr int kThreads = 256;
constexpr int kWarps = kThreads / 32;

struct Code {
    uint32_t code[ENTRO_MAX_SYMBOLS];
    uint8_t len[ENTRO_MAX_SYMBOLS];
};

constexpr uint32_t kGroup = 8;    // symbols per group

// Calls f(symbol) for every symbol of sub-block `lane` of the chunk that starts at element
// `first` and holds m symbols, in stored order.
template <class F>
__device__ __forceinline__ void for_each_symbol(const uint8_t* __restrict__ q, uint64_t first, uint32_t m,
                                                uint32_t lane, F f)
{
    for (uint32_t g = lane; g * kGroup < m; g += kSubBlocks) {
        const uint32_t base = g * kGroup;
        if (base + kGroup <= m) {
            const uint2 v = *reinterpret_cast<const uint2*>(q + first + base);   // q is 16-byte aligned, base a multiple of 8
#pragma unroll
            for (int k = 0; k < 4; ++k) f((v.x >> (8 * k)) & 0xffu);
#pragma unroll
            for (int k = 0; k < 4; ++k) f((v.y >> (8 * k)) & 0xffu);
        } else {
            for (uint32_t k = base; k < m; ++k) f((uint32_t)q[first + k]);
        }
    }
}

// Pass 1: one warp per chunk, one lane per sub-block.
__global__ void __launch_bounds__(kThreads) sub_lengths_kernel(const uint8_t* __restrict__ q, uint64_t n,
                                                               uint32_t chunk_symbols, uint32_t n_chunks,
                                                               const Code* __restrict__ cb,
                                                               uint16_t* __restrict__ sub_len,
                                                               unsigned long long* __restrict__ chunk_bits,
                                                               uint32_t* __restrict__ bad_symbol)
{
    __shared__ uint8_t s_len[ENTRO_MAX_SYMBOLS];
    for (int i = threadIdx.x; i < ENTRO_MAX_SYMBOLS; i += kThreads) s_len[i] = cb->len[i];
    __syncthreads();
    const uint32_t lane = threadIdx.x & 31;
    for (uint32_t c = blockIdx.x * kWarps + (threadIdx.x >> 5); c < n_chunks; c += gridDim.x * kWarps) {
        const uint64_t first = (uint64_t)c * chunk_symbols;
        const uint32_t m = (uint32_t)min((uint64_t)chunk_symbols, n - first);
        uint32_t bits = 0, bad = 0;
        for_each_symbol(q, first, m, lane, [&](uint32_t sym) {
            uint32_t l = s_len[sym];
            bad |= (l == 0);
            bits += l;
        });
        if (bad) atomicOr(bad_symbol, 1u);
        sub_len[(uint64_t)c * kSubBlocks + lane] = (uint16_t)bits;
        uint32_t total = bits;
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) total += __shfl_xor_sync(0xffffffffu, total, d);
        if (lane == 0) chunk_bits[c] = total;
    }
}

// Pass 2: exclusive prefix sum of the chunk lengths by one block; offsets[n_chunks] = total.
__global__ void __launch_bounds__(1024) chunk_offsets_kernel(const unsigned long long* __restrict__ chunk_bits,
                                                             uint32_t n_chunks,
                                                             unsigned long long* __restrict__ offsets)
{
    __shared__ unsigned long long warp_sum[32];
    __shared__ unsigned long long carry;
    if (threadIdx.x == 0) carry = 0;
    __syncthreads();
    const uint32_t lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    for (uint32_t base = 0; base < n_chunks; base += 1024) {
        uint32_t i = base + threadIdx.x;
        unsigned long long v = i < n_chunks ? chunk_bits[i] : 0ull;
        unsigned long long incl = v;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            unsigned long long t = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= (uint32_t)d) incl += t;
        }
        if (lane == 31) warp_sum[warp] = incl;
        __syncthreads();
        if (warp == 0) {
            unsigned long long w = warp_sum[lane];
            unsigned long long wi = w;
#pragma unroll
            for (int d = 1; d < 32; d <<= 1) {
                unsigned long long t = __shfl_up_sync(0xffffffffu, wi, d);
                if (lane >= (uint32_t)d) wi += t;
            }
            warp_sum[lane] = wi - w;  // exclusive
        }
        __syncthreads();
        unsigned long long excl = carry + warp_sum[warp] + incl - v;
        if (i < n_chunks) offsets[i] = excl;
        __syncthreads();
        if (threadIdx.x == 1023) carry = excl + v;
        __syncthreads();
    }
    if (threadIdx.x == 0) offsets[n_chunks] = carry;
}

// Pass 3: one warp per chunk; every lane writes the bits of its own sub-block.  Words that
// a sub-block shares with a neighbour are merged with atomicOr into the zeroed stream.
__global__ void __launch_bounds__(kThreads) pack_kernel(const uint8_t* __restrict__ q, uint64_t n,
                                                        uint32_t chunk_symbols, uint32_t n_chunks,
                                                        const Code* __restrict__ cb,
                                                        const unsigned long long* __restrict__ offsets,
                                                        const uint16_t* __restrict__ sub_len,
                                                        uint32_t* __restrict__ stream, uint64_t stream_words,
                                                        unsigned long long* __restrict__ report)
{
    // report (batched calls): [0] total bits, [1] != 0 if they do not fit stream_words words (then
    // nothing is written)
    if (report) {
        const unsigned long long total = offsets[n_chunks];
        const bool fits = (total + 31) / 32 <= stream_words;
        if (blockIdx.x == 0 && threadIdx.x == 0) {
            report[0] = total;
            report[1] = fits ? 0ull : 1ull;
        }
        if (!fits) return;
    }
    __shared__ uint32_t s_code[ENTRO_MAX_SYMBOLS];
    __shared__ uint8_t s_len[ENTRO_MAX_SYMBOLS];
    for (int i = threadIdx.x; i < ENTRO_MAX_SYMBOLS; i += kThreads) {
        s_code[i] = cb->code[i];
        s_len[i] = cb->len[i];
    }
    __syncthreads();
    const uint32_t lane = threadIdx.x & 31;
    for (uint32_t c = blockIdx.x * kWarps + (threadIdx.x >> 5); c < n_chunks; c += gridDim.x * kWarps) {
        uint32_t mine = sub_len[(uint64_t)c * kSubBlocks + lane];
        uint32_t incl = mine;
#pragma unroll
        for (int d = 1; d < 32; d <<= 1) {
            uint32_t t = __shfl_up_sync(0xffffffffu, incl, d);
            if (lane >= (uint32_t)d) incl += t;
        }
        unsigned long long pos = offsets[c] + (incl - mine);   // first bit of this sub-block
        const uint64_t first = (uint64_t)c * chunk_symbols;
        const uint32_t m = (uint32_t)min((uint64_t)chunk_symbols, n - first);
        if (lane * kGroup >= m) continue;     // empty sub-block

        // acc holds `fill` pending bits, left-justified; word is where they go next.
        unsigned long long word = pos >> 5;
        uint32_t fill = (uint32_t)(pos & 31);   // bits of `word` that belong to earlier sub-blocks
        unsigned long long acc = 0;             // bits [63 - fill ...] downwards are ours
        bool first_word = true;
        for_each_symbol(q, first, m, lane, [&](uint32_t sym) {
            uint32_t l = s_len[sym];
            if (l == 0) return;                 // reported by pass 1
            acc |= (unsigned long long)s_code[sym] << (64 - fill - l);
            fill += l;
            if (fill >= 32) {
                uint32_t out = (uint32_t)(acc >> 32);
                if (first_word) atomicOr(&stream[word], out);
                else stream[word] = out;
                first_word = false;
                ++word;
                acc <<= 32;
                fill -= 32;
            }
        });
        if (fill) atomicOr(&stream[word], (uint32_t)(acc >> 32));
    }
}

}  // namespace
}  // namespace entro

using namespace entro;

extern "C" entro_status entro_encode(const uint8_t* q_dev, uint64_t n, const entro_codebook* cb,
                                     uint32_t chunk_symbols, uint32_t* stream_dev, uint64_t stream_cap_words,
                                     void* index_dev, uint64_t index_cap_bytes, uint64_t* total_bits_host,
                                     void* cuda_stream)
{
    if (!q_dev || !cb || !stream_dev || !index_dev || !total_bits_host || n == 0) return ENTRO_ERR_INVALID_ARG;
    if (chunk_symbols < kSubBlocks || chunk_symbols % kSubBlocks || chunk_symbols > ENTRO_MAX_CHUNK_SYMBOLS)
        return ENTRO_ERR_INVALID_ARG;
    // q is read as 8-byte vectors (a group of eight symbols at a time)
    if (!aligned(q_dev, 16) || !aligned(stream_dev, 16) || !aligned(index_dev, 8)) return ENTRO_ERR_INVALID_ARG;
    if (!codebook_lengths_valid(cb)) return ENTRO_ERR_INVALID_ARG;
    const uint64_t nc64 = num_chunks(n, chunk_symbols);
    if (nc64 > 0x7fffffffull) return ENTRO_ERR_UNSUPPORTED;
    const uint32_t nc = (uint32_t)nc64;
    if (entro_index_bytes(n, chunk_symbols) > index_cap_bytes) return ENTRO_ERR_BUFFER_TOO_SMALL;
    if (stream_cap_words <= ENTRO_STREAM_SLACK_WORDS) return ENTRO_ERR_BUFFER_TOO_SMALL;

    Guard g;
    Workspace* ws = workspace();
    if (!ws) return ENTRO_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)cuda_stream;

    // workspace: [Code][chunk_bits: nc u64][flag]
    const size_t code_bytes = (sizeof(Code) + 15) & ~(size_t)15;
    const size_t need = code_bytes + (size_t)nc * 8 + 16;
    if (!reserve_device(ws, need) || !reserve_pinned(ws, code_bytes + 16)) return ENTRO_ERR_CUDA;
    Code* host_code = static_cast<Code*>(ws->pinned);
    for (int k = 0; k < ENTRO_MAX_SYMBOLS; ++k) {
        host_code->code[k] = k < cb->nsym ? cb->code[k] : 0;
        host_code->len[k] = k < cb->nsym ? cb->len[k] : 0;
    }
    char* base = static_cast<char*>(ws->dev);
    Code* dev_code = reinterpret_cast<Code*>(base);
    unsigned long long* chunk_bits = reinterpret_cast<unsigned long long*>(base + code_bytes);
    uint32_t* flag = reinterpret_cast<uint32_t*>(base + code_bytes + (size_t)nc * 8);
    unsigned long long* offsets = static_cast<unsigned long long*>(index_dev);
    uint16_t* sub_len = reinterpret_cast<uint16_t*>(offsets + nc + 1);

    ENTRO_CUDA(cudaMemcpyAsync(dev_code, host_code, sizeof(Code), cudaMemcpyHostToDevice, s));
    mark_pinned_in_use(ws, s);
    ENTRO_CUDA(cudaMemsetAsync(flag, 0, 16, s));
    int grid = (int)((nc + kWarps - 1) / kWarps);
    int cap = ws->sm_count * 8;
    if (grid > cap) grid = cap;
    sub_lengths_kernel<<<grid, kThreads, 0, s>>>(q_dev, n, chunk_symbols, nc, dev_code, sub_len, chunk_bits, flag);
    chunk_offsets_kernel<<<1, 1024, 0, s>>>(chunk_bits, nc, offsets);
    count_launch(2);
    ENTRO_CUDA(cudaGetLastError());

    // total bits and the bad-symbol flag decide whether the pack pass may run
    struct { unsigned long long total; uint32_t bad; uint32_t pad; } h;
    ENTRO_CUDA(cudaMemcpyAsync(&h.total, offsets + nc, 8, cudaMemcpyDeviceToHost, s));
    ENTRO_CUDA(cudaMemcpyAsync(&h.bad, flag, 4, cudaMemcpyDeviceToHost, s));
    ENTRO_CUDA(cudaStreamSynchronize(s));
    if (h.bad) return ENTRO_ERR_INVALID_ARG;
    const uint64_t words = (h.total + 31) / 32;
    if (words + ENTRO_STREAM_SLACK_WORDS > stream_cap_words) return ENTRO_ERR_BUFFER_TOO_SMALL;

    ENTRO_CUDA(cudaMemsetAsync(stream_dev, 0, stream_cap_words * sizeof(uint32_t), s));
    pack_kernel<<<grid, kThreads, 0, s>>>(q_dev, n, chunk_symbols, nc, dev_code, offsets, sub_len, stream_dev, 0, nullptr);
    count_launch();
    ENTRO_CUDA(cudaGetLastError());
    ENTRO_CUDA(cudaStreamSynchronize(s));
    *total_bits_host = h.total;
    return ENTRO_OK;
}

// The same for many tensors with one synchronisation at the end: per tensor the three passes
// are queued back to back, the pack pass itself refuses to write a stream that would not fit,
// and totals and error flags of all tensors come back in one copy.
extern "C" entro_status entro_encode_batched(const entro_encode_job* jobs, int njobs, uint64_t* total_bits_host,
                                             void* cuda_stream)
{
    if (njobs < 0 || (njobs > 0 && (!jobs || !total_bits_host))) return ENTRO_ERR_INVALID_ARG;
    if (njobs == 0) return ENTRO_OK;
    uint32_t max_nc = 0;
    for (int j = 0; j < njobs; ++j) {
        const entro_encode_job& job = jobs[j];
        if (!job.q_dev || !job.cb_host || !job.stream_dev || !job.index_dev || job.n == 0) return ENTRO_ERR_INVALID_ARG;
        if (job.chunk_symbols < kSubBlocks || job.chunk_symbols % kSubBlocks || job.chunk_symbols > ENTRO_MAX_CHUNK_SYMBOLS)
            return ENTRO_ERR_INVALID_ARG;
        if (!aligned(job.q_dev, 16) || !aligned(job.stream_dev, 16) || !aligned(job.index_dev, 8)) return ENTRO_ERR_INVALID_ARG;
        if (!codebook_lengths_valid(job.cb_host)) return ENTRO_ERR_INVALID_ARG;
        const uint64_t nc64 = num_chunks(job.n, job.chunk_symbols);
        if (nc64 > 0x7fffffffull) return ENTRO_ERR_UNSUPPORTED;
        if (entro_index_bytes(job.n, job.chunk_symbols) > job.index_cap_bytes) return ENTRO_ERR_BUFFER_TOO_SMALL;
        if (job.stream_cap_words <= ENTRO_STREAM_SLACK_WORDS) return ENTRO_ERR_BUFFER_TOO_SMALL;
        if ((uint32_t)nc64 > max_nc) max_nc = (uint32_t)nc64;
    }
    Guard g;
    Workspace* ws = workspace();
    if (!ws) return ENTRO_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    // device area: [Code x njobs][report x njobs: total, overflow][bad-symbol flag x njobs][chunk bits of the tensor in flight]
    const size_t code_bytes = (sizeof(Code) + 15) & ~(size_t)15;
    const size_t codes_bytes = code_bytes * (size_t)njobs;
    const size_t report_bytes = (size_t)njobs * 16;
    const size_t flags_bytes = ((size_t)njobs * 4 + 15) & ~(size_t)15;
    if (!reserve_device(ws, codes_bytes + report_bytes + flags_bytes + (size_t)max_nc * 8 + 16)) return ENTRO_ERR_CUDA;
    if (!reserve_pinned(ws, codes_bytes + report_bytes + flags_bytes)) return ENTRO_ERR_CUDA;
    char* base = static_cast<char*>(ws->dev);
    char* host = static_cast<char*>(ws->pinned);
    for (int j = 0; j < njobs; ++j) {
        Code* hc = reinterpret_cast<Code*>(host + code_bytes * (size_t)j);
        const entro_codebook* cb = jobs[j].cb_host;
        for (int k = 0; k < ENTRO_MAX_SYMBOLS; ++k) {
            hc->code[k] = k < cb->nsym ? cb->code[k] : 0;
            hc->len[k] = k < cb->nsym ? cb->len[k] : 0;
        }
    }
    unsigned long long* report = reinterpret_cast<unsigned long long*>(base + codes_bytes);
    uint32_t* flags = reinterpret_cast<uint32_t*>(base + codes_bytes + report_bytes);
    unsigned long long* chunk_bits = reinterpret_cast<unsigned long long*>(base + codes_bytes + report_bytes + flags_bytes);
    ENTRO_CUDA(cudaMemcpyAsync(base, host, codes_bytes, cudaMemcpyHostToDevice, s));
    ENTRO_CUDA(cudaMemsetAsync(report, 0, report_bytes + flags_bytes, s));
    for (int j = 0; j < njobs; ++j) {
        const entro_encode_job& job = jobs[j];
        const uint32_t nc = (uint32_t)num_chunks(job.n, job.chunk_symbols);
        const Code* dev_code = reinterpret_cast<const Code*>(base + code_bytes * (size_t)j);
        unsigned long long* offsets = static_cast<unsigned long long*>(job.index_dev);
        uint16_t* sub_len = reinterpret_cast<uint16_t*>(offsets + nc + 1);
        int grid = (int)((nc + kWarps - 1) / kWarps);
        const int cap = ws->sm_count * 8;
        if (grid > cap) grid = cap;
        sub_lengths_kernel<<<grid, kThreads, 0, s>>>(job.q_dev, job.n, job.chunk_symbols, nc, dev_code, sub_len, chunk_bits, flags + j);
        chunk_offsets_kernel<<<1, 1024, 0, s>>>(chunk_bits, nc, offsets);
        ENTRO_CUDA(cudaMemsetAsync(job.stream_dev, 0, job.stream_cap_words * sizeof(uint32_t), s));
        pack_kernel<<<grid, kThreads, 0, s>>>(job.q_dev, job.n, job.chunk_symbols, nc, dev_code, offsets, sub_len, job.stream_dev,
                                              job.stream_cap_words - ENTRO_STREAM_SLACK_WORDS, report + 2 * (size_t)j);
        count_launch(3);
    }
    ENTRO_CUDA(cudaGetLastError());
    char* host_report = host + codes_bytes;                 // behind the codes, which the device may still be reading
    ENTRO_CUDA(cudaMemcpyAsync(host_report, report, report_bytes + flags_bytes, cudaMemcpyDeviceToHost, s));
    ENTRO_CUDA(cudaStreamSynchronize(s));
    const unsigned long long* hr = reinterpret_cast<const unsigned long long*>(host_report);
    const uint32_t* hf = reinterpret_cast<const uint32_t*>(host_report + report_bytes);
    entro_status st = ENTRO_OK;
    for (int j = 0; j < njobs; ++j) {
        total_bits_host[j] = hr[2 * j];
        if (hf[j]) st = ENTRO_ERR_INVALID_ARG;                       // a symbol without a code
        else if (hr[2 * j + 1] && st == ENTRO_OK) st = ENTRO_ERR_BUFFER_TOO_SMALL;
    }
    return st;
}
