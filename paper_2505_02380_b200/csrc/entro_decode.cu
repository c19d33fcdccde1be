// Parallel Huffman decode fused with dequantisation to fp16 (Section 3, "Segmentation for
// parallel Huffman decoding"; Eq. 1 inverted).  This file: the persistent kernel, its launch
// and the entry points; entro_decode_{common,tables,reader,chunk}.cuh hold the device parts.
//
// Work split: a chunk (one segment) is decoded by one warp, each lane owning one of the
// chunk's 32 sub-blocks.  The lanes' start positions come from a warp prefix sum over the
// sub-block bit lengths stored in the index.  A persistent grid pulls work items (runs of
// chunks of one tensor) from a global counter; the warps of a CTA share out an item's
// chunks through a shared-memory counter.  Every warp runs a three-deep pipeline: while it
// decodes chunk i, the bytes of chunk i + 1 are arriving in its shared-memory ring through
// one bulk asynchronous copy, and the index entries of chunk i + 2 are on their way into
// a shared-memory slot of the warp.  Lanes walk their bits with lookup tables whose entries already hold the
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
#include <cstring>
#include <new>

#include "entro_decode_chunk.cuh"

namespace entro {
namespace {

// ------------------------------------------------------------------ persistent kernel

// n 16-byte words from global to shared memory by the whole CTA, four reads in flight per
// thread before the first store (one round trip to L2 per four words instead of one per word).
__device__ __forceinline__ void copy_in(uint4* dst, const uint4* __restrict__ src, uint32_t n)
{
    for (uint32_t base = threadIdx.x; base < n; base += 4u * blockDim.x) {
        uint4 v[4];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t i = base + (uint32_t)k * blockDim.x;
            v[k] = i < n ? __ldg(src + i) : make_uint4(0u, 0u, 0u, 0u);
        }
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            const uint32_t i = base + (uint32_t)k * blockDim.x;
            if (i < n) dst[i] = v[k];
        }
    }
}

// The exponent-indexed table of a tensor into the first 64 KB of shared memory: cell-major
// copies, word w holds cell w / copies.
__device__ __forceinline__ void load_exp_table(const TensorTables* tt, uint32_t expm)
{
    const uint32_t shift = 9u - expm;                        // log2 of the number of copies
    if (shift >= 2u) {
        // four or more copies: the four words of a 16-byte store belong to one cell.  Four reads
        // are in flight per thread before the first store (one round trip to L2 instead of four).
        uint4* s4 = reinterpret_cast<uint4*>(smem);
        constexpr uint32_t kQuads = (uint32_t)kExpEntriesMax / 4u;
        for (uint32_t base = threadIdx.x; base < kQuads; base += 4u * blockDim.x) {
            uint32_t v[4];
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint32_t q = base + (uint32_t)k * blockDim.x;
                v[k] = q < kQuads ? __ldg(tt->exp_lut() + ((4u * q) >> shift)) : 0u;
            }
#pragma unroll
            for (int k = 0; k < 4; ++k) {
                const uint32_t q = base + (uint32_t)k * blockDim.x;
                if (q < kQuads) s4[q] = make_uint4(v[k], v[k], v[k], v[k]);
            }
        }
    } else {
        uint32_t* s1 = reinterpret_cast<uint32_t*>(smem);
        for (uint32_t w = threadIdx.x; w < (uint32_t)kExpEntriesMax; w += blockDim.x)
            s1[w] = __ldg(tt->exp_lut() + (w >> shift));
    }
}

// A CTA calls this once, after its last claim of a work item.  The last CTA of the grid to get
// here puts the work counter and the count of finished CTAs back to zero.
__device__ __forceinline__ void cta_finished(uint32_t* control)
{
    if (atomicAdd(control + 2, 1u) == gridDim.x - 1u) {
        control[0] = 0;
        control[2] = 0;
    }
}

// Tensor of a work item: the last t with item_start[t] <= item, found by a whole warp, each
// lane reading one of 32 evenly spaced entries per round (two dependent reads for up to 1024
// tensors, where a binary search by one thread takes ten).  All lanes return the same t.
__device__ __forceinline__ uint32_t tensor_of_item(const uint32_t* __restrict__ item_start, uint32_t ntensors, uint32_t item,
                                                   uint32_t lane)
{
    uint32_t lo = 0, n = ntensors;
    while (n > 1u) {
        const uint32_t step = (n + 31u) >> 5;
        const uint32_t at = lo + lane * step;
        const uint32_t v = at < lo + n ? __ldg(item_start + at) : 0xffffffffu;
        const uint32_t k = (uint32_t)__popc(__ballot_sync(0xffffffffu, v <= item));   // >= 1: item_start[lo] <= item
        const uint32_t end = lo + n;
        lo += (k - 1u) * step;
        n = min(step, end - lo);
    }
    return lo;
}

// item_start[t] = first work item of tensor t, item_start[ntensors] = number of items; an
// item is up to tensors[t].item_chunks consecutive chunks of one tensor.
// kSink says where the decoded values go.  With kSinkGemv they are not stored: gemv[t]
// describes the matrix-vector products they enter (the fused decode + dequantise + GEMV of a
// token step, one token or a small batch).
// control: [0] the work counter, which must be 0 at the start and is 0 again at the end (the
// last CTA to finish puts it back, so that a prepared launch can be repeated with nothing in
// between), [1] the status word, [2] CTAs that have finished.
template <int K, int kSink>
__global__ void __launch_bounds__(1024, 1) decode_kernel(const DevTensor* __restrict__ tensors, int ntensors,
                                                         const uint32_t* __restrict__ item_start,
                                                         const TensorTables* __restrict__ tables,
                                                         uint32_t stage_bytes,
                                                         uint32_t* __restrict__ control,
                                                         const GemvTensor* __restrict__ gemv, uint32_t rings_at,
                                                         uint32_t striped)
{
    constexpr int kBatch = kGemvBatchOf<kSink>;
    constexpr bool kGemv = kBatch > 0;
    // layout: [tables][aux][tensor]([gemv descriptor][x])[per-warp rings][over-read pad][mbarriers][index slots][item slots]
    if (smem_addr(smem) != kSmemBase) {   // the lookups' address arithmetic would be wrong: refuse to run
        if (threadIdx.x == 0) {
            atomicOr(control + 1, kStatInternal);
            cta_finished(control);
        }
        return;
    }
    DecodeAux* s_aux = aux_ptr<K>();
    DevTensor* s_tensor = tensor_ptr<K>();
    const uint32_t warps = blockDim.x >> 5;
    const uint32_t warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const uint32_t kRings = rings_at;          // rings_offset<K>(kGemv, bytes of staged x)
    const uint32_t after = kRings + warps * stage_bytes + kOverRead;          // offset in smem, a multiple of 16
    const uint32_t slots = after + warps * 16u;
    volatile uint32_t* s_item = reinterpret_cast<volatile uint32_t*>(smem + slots + warps * 2u * kSlotBytes);   // [4]
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

    // s_item[slot] = the item's number within its tensor, s_item[2 + slot] = the tensor, or kNone
    // when the items have run out.  Warp 0 puts the next item on record, tensor included, before
    // the barrier that ends the current one, so nobody reads global memory behind that barrier
    // to find out where to go on.
    const uint32_t total_items = item_start[ntensors];
    // The first `striped` items (a multiple of the grid size, all of full size) are claimed in
    // an order that hands a CTA consecutive items of the list, hence mostly of one tensor, as long
    // as the CTAs keep pace: claim i is item (i mod grid) * rows + i / grid.  The table is then
    // reloaded a few times per CTA instead of once per item.  The graded items at the end keep
    // their order, so the CTAs still finish together.
    const uint32_t stripe_rows = striped / gridDim.x;
    auto put_on_record = [&](uint32_t item, uint32_t where) {      // warp 0, all lanes, the same item
        uint32_t t = kNone, rel = 0;
        if (item < striped) item = (item % gridDim.x) * stripe_rows + item / gridDim.x;
        if (item < total_items) {
            t = tensor_of_item(item_start, (uint32_t)ntensors, item, lane);
            rel = item - __ldg(item_start + t);
        }
        if (lane == 0) {
            s_item[where] = rel;
            s_item[2u + where] = t;
        }
    };
    if (warp == 0) {
        uint32_t item0 = 0;
        if (lane == 0) item0 = atomicAdd(control, 1u);
        put_on_record(__shfl_sync(0xffffffffu, item0, 0), 0u);
    }
    __syncthreads();
    int cur = -1;
    uint32_t slot = 0;
    while (true) {
        const uint32_t item_tensor = s_item[2u + slot];
        if (item_tensor == kNone) break;
        const uint32_t item_rel = s_item[slot];
        // claim the next item early; the answer of the global counter is not waited for here
        // but put on record when this item is done, before the barrier that ends it
        uint32_t next_item = 0;
        if (threadIdx.x == 0) next_item = atomicAdd(control, 1u);
        const int lo = (int)item_tensor;
        if (lo != cur) {
            cur = lo;
            const TensorTables* tt = tables + cur;
            // (both flags are read at once and first: the table's reads start one round trip after the switch)
            const uint32_t is_oct = __ldg(&tt->aux.oct), expm = __ldg(&tt->aux.expm);
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
            if (is_oct) {
                copy_in(reinterpret_cast<uint4*>(smem), tt->oct_val, 1u << K);
                const uint4* g2 = reinterpret_cast<const uint4*>(tt->oct_len);
                uint4* s2 = reinterpret_cast<uint4*>(smem + (16u << K));
                for (uint32_t i = threadIdx.x; i < (1u << K) / 16; i += blockDim.x) s2[i] = __ldg(g2 + i);
                uint32_t* s3 = reinterpret_cast<uint32_t*>(smem + (17u << K));
                for (uint32_t i = threadIdx.x; i < (uint32_t)kExpEntriesMin; i += blockDim.x) s3[i] = __ldg(tt->exp_small + i);
            } else {
                load_exp_table(tt, expm);
            }
            __syncthreads();
        }
        const DevTensor& T = *s_tensor;
        const uint32_t first = item_rel * T.item_chunks;
        const uint32_t count = min(T.item_chunks, T.n_chunks - first);   // chunks of this item

        // The warps deal out the item's chunks among themselves, warp w taking chunks w, w + warps,
        // ... of the item (the chunks of one tensor cost about the same, so nobody waits long at the
        // item's end).  Each warp, per turn: start the bulk copy of chunk i + 1 (its offsets arrived
        // a turn ago), work out the lanes' positions in chunk i, ask for the index entries of chunk
        // i + 2 in the slot that frees, decode chunk i.
        uint32_t upcoming = first + warp;           // the warp's next chunk whose index entries have not been asked for
        const uint32_t item_end = first + count;
        auto next_chunk = [&]() -> uint32_t {
            const uint32_t c = upcoming < item_end ? upcoming : kNone;
            upcoming += warps;
            return c;
        };
        Ready r0;
        r0.c = kNone;
        r0.meta = ready_meta(0, 0, 0, kSkip);
        const uint32_t turns = s_aux->turns;
        const uint32_t both_slots = 2u * cx.idx_addr + kSlotBytes;   // the sum of the two slots' addresses
        uint32_t sp = cx.idx_addr;                  // slot of the chunk fetched last
        uint32_t c2 = next_chunk();
        fetch_index(s_aux, T, c2, sp, lane);
        while (true) {
            Ready r1 = prepare(cx, T, turns, stage_bytes, status, c2, sp, r0, lane);
            const uint32_t other = both_slots - sp;
            const Lane L = decode_start<K>(cx, status, r0, other, lane);
            __syncwarp();                           // every lane has read the slot before it is refilled
            c2 = r1.c == kNone ? kNone : next_chunk();
            fetch_index(s_aux, T, c2, other, lane);
            decode_finish<K, kSink>(cx, status, r0, L, lane, stage_bytes);
            if (r1.c == kNone) break;
            // the ring is free now: a copy that had to wait for it starts here, a turn's worth of
            // bookkeeping before its bytes are asked for (its offset is still in the chunk's slot)
            if (r1.kind() == kStaged && !r1.issued()) issue_copy(cx, T, r1, (lds64(sp + 64u) >> 3) & ~15ull, lane, stage_bytes);
            r0 = r1;
            sp = other;
        }
        asm volatile("cp.async.wait_all;" ::: "memory");
        if (warp == 0) put_on_record(__shfl_sync(0xffffffffu, next_item, 0), slot ^ 1u);
        __syncthreads();   // tables may be replaced; the next item's record is now visible
        slot ^= 1u;
    }
    // A warp that gave up on a bulk copy lets it land (bounded) before its buffer goes away.
    const uint32_t issued = cx.state & 0x7fffffffu;
    if (cx.dead() && issued) (void)mbar_wait(cx.bar + 8u * ((issued - 1) & 1u), ((issued - 1) >> 1) & 1u);
    if (threadIdx.x == 0) cta_finished(control);
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
        tensors, ntensors, item_start, tables, sh.stage_bytes, ws->control, gemv, rings_offset<K>(kGemv, x_bytes),
        ws->big_items / grid * grid);
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
    uint32_t base = 0, tail = 0, unit = 32;
    bool graded = false;
    uint64_t items = 0;        // work items of the tensors planned so far
    uint64_t big_items = 0;    // of those, the ones before the first tensor with graded (small) items
    bool tail_seen = false;
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
    uint64_t want = (p.total + ctas * 5 - 1) / (ctas * 5);
    p.unit = (uint32_t)cfg.warps_per_cta;
    // fewer chunks than warps on the GPU: items of two chunks, so that the launch spreads over as
    // many SMs as it can (a lone warp decodes a chunk several times faster than one of 32 on an SM)
    if (p.total < ctas * (uint64_t)cfg.warps_per_cta) p.unit = 2;
    want = (want + p.unit - 1) / p.unit * p.unit;
    if (want < (uint64_t)p.unit) want = p.unit;
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
    t.last_bit = d.stream_words * 4 >= 28 ? (d.stream_words * 4 - 28) * 8 + 7 : 0;
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
    if (per_item < plan.unit) per_item = plan.unit;
    // the tensor's items of equal size (a short last item leaves most of a CTA's warps idle),
    // whole rounds of the 32 warps
    const uint64_t pieces = (nc + per_item - 1) / per_item;
    if (pieces > 1) per_item = (uint32_t)(((nc + pieces - 1) / pieces + plan.unit - 1u) / plan.unit * plan.unit);
    t.item_chunks = per_item;
    plan.seen += nc;
    t.raw_symbols = 0;
    t.full_chunks = (uint32_t)(d.n / d.chunk_symbols);
    t.pad[0] = t.pad[1] = 0;
    for (int j = 0; j < ENTRO_MAX_SYMBOLS; ++j) t.len[j] = j < d.cb.nsym ? d.cb.len[j] : 0;
    const uint64_t n_items = (nc + t.item_chunks - 1) / t.item_chunks;
    const bool small = plan.graded && (plan.seen * 100 > plan.total * 88);     // (seen already includes this tensor)
    plan.items += n_items;
    if (small) plan.tail_seen = true;
    if (!plan.tail_seen) plan.big_items = plan.items;
    return n_items;
}

}  // namespace

// A chunk is decoded from shared memory only if its bytes fit the warp's ring; otherwise its
// lanes read global memory word by word, about six times slower.  Where most of a launch's
// symbols sit in chunks that (going by the streams' sizes) do not fit the ring of the
// configured shape, the launch runs with half or a quarter of the warps and accordingly
// larger rings: slower per SM than the full shape, but far better than the fallback.
DecodeConfig config_for(const DecodeConfig& base, const entro_tensor_desc* descs, int ntensors, int max_smem)
{
    DecodeConfig cfg = base;
    for (int step = 0; step < 2; ++step) {
        const Shape sh = shape_for(cfg, max_smem);
        if (sh.stage_bytes == 0 || cfg.warps_per_cta < 16) break;
        uint64_t total = 0, too_big = 0;
        for (int i = 0; i < ntensors; ++i) {
            const entro_tensor_desc& d = descs[i];
            if (!d.chunk_symbols || d.n < d.chunk_symbols || d.stream_words < ENTRO_STREAM_SLACK_WORDS)
                continue;                             // nothing, or only a ragged chunk (general path anyway), or not valid
            total += d.n;
            const uint64_t stream_bytes = (d.stream_words - ENTRO_STREAM_SLACK_WORDS) * 4;
            const uint64_t chunk_bytes = stream_bytes * d.chunk_symbols / d.n + 48;   // mean chunk, margins of the copy
            if (chunk_bytes > sh.stage_bytes) too_big += d.n;
        }
        if (too_big * 2 <= total) break;
        cfg.warps_per_cta /= 2;
    }
    return shape_for(cfg, max_smem).stage_bytes ? cfg : base;
}

// Upload descriptors, build the tables and run the persistent decode kernel.
entro_status decode_batched_locked(Workspace* ws, const entro_tensor_desc* descs, int ntensors, cudaStream_t s,
                                   int sink = kSinkFp16)
{
    const DecodeConfig cfg = config_for(decode_config(), descs, ntensors, ws->max_smem_optin);
    int live = 0;
    for (int i = 0; i < ntensors; ++i) {
        entro_status st = validate_desc(descs[i]);
        if (st != ENTRO_OK) return st;
        if (descs[i].n) live++;
    }
    if (live == 0) return ENTRO_OK;

    // A repeat of the last call (few tensors, the very same descriptors, launch shape and
    // sink, nothing else in the device area since): descriptors and tables are still in place,
    // and the work counter is back at zero, so the decode launch is all there is to do.  (Tables
    // are constants of a compressed tensor; only the choice of the decode mode looks at the
    // device, at the stream's bit rate, and every mode decodes every stream.)
    const bool few = ntensors <= Workspace::kKeptTensors;
    if (few && ws->kept && ws->kept_ntensors == ntensors && ws->kept_sink == sink &&
        memcmp(&ws->kept_cfg, &cfg, sizeof(cfg)) == 0 &&
        memcmp(ws->kept_descs, descs, (size_t)ntensors * sizeof(entro_tensor_desc)) == 0) {
        char* kept_base = static_cast<char*>(ws->dev);
        const size_t kept_tensors_bytes = (size_t)ws->kept_live * sizeof(DevTensor);
        const size_t kept_upload = kept_tensors_bytes + ((((size_t)ws->kept_live + 1) * 4 + 15) & ~(size_t)15);
        return launch_decode_any(ws, cfg, reinterpret_cast<DevTensor*>(kept_base), ws->kept_live,
                                 reinterpret_cast<uint32_t*>(kept_base + kept_tensors_bytes), ws->kept_items,
                                 reinterpret_cast<TensorTables*>(kept_base + kept_upload), s, nullptr, sink);
    }
    ItemPlan plan = plan_items(cfg, descs, ntensors, ws->sm_count);

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
    build_tables_kernel<<<dim3((unsigned)live, table_slices(live, ws->sm_count)), 256, 0, s>>>(dt, cfg.lut_bits, dtables, ws->control, nullptr);
    count_launch();
    ENTRO_CUDA(cudaGetLastError());
    // Striped claims pay where decoding is bound by instructions (8-bit alphabets: fewer table
    // reloads); a launch of 4-bit alphabets runs near the HBM peak and loses by them (148 places
    // written at once instead of neighbouring ones: 2.50 against 2.465 ms on the mistral-shaped model).
    uint64_t wide_symbols = 0, all_symbols = 0;
    for (int i = 0; i < ntensors; ++i) {
        all_symbols += descs[i].n;
        if (descs[i].cb.nsym > 16) wide_symbols += descs[i].n;
    }
    ws->big_items = (plan.graded && !few && wide_symbols * 2 > all_symbols) ? (uint32_t)plan.big_items : 0u;
    const entro_status st = launch_decode_any(ws, cfg, dt, live, ditems, (uint32_t)items, dtables, s, nullptr, sink);
    ws->big_items = 0;
    if (few && st == ENTRO_OK) {
        ws->kept = true;
        ws->kept_ntensors = ntensors;
        ws->kept_live = live;
        ws->kept_sink = sink;
        ws->kept_items = (uint32_t)items;
        ws->kept_cfg = cfg;
        memcpy(ws->kept_descs, descs, (size_t)ntensors * sizeof(entro_tensor_desc));
    }
    return st;
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
        if (!io[i].stream_host || !io[i].index_host) return ENTRO_ERR_INVALID_ARG;
        entro_status st = validate_desc(descs[i]);
        if (st != ENTRO_OK) return st;
        out_bytes += descs[i].n * 2;
    }
    Guard g;
    Workspace* ws = workspace();
    if (!ws || !copy_streams_ready(ws)) return ENTRO_ERR_CUDA;
    // groups of consecutive tensors, about equal in output bytes
    const uint64_t per_group = out_bytes / Workspace::kCopyGroups + 1;
    auto enqueue = [&]() -> entro_status {
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
                if (!d.n || !io[i].out_fp16_host) continue;     // no host buffer: the result stays on the device
                ENTRO_CUDA(cudaMemcpyAsync(io[i].out_fp16_host, d.out_fp16_dev, d.n * 2, cudaMemcpyDeviceToHost, ws->copy_out));
            }
            first = last;
            ++group;
        }
        ENTRO_CUDA(cudaEventRecord(ws->ev_edge, ws->copy_out));
        ENTRO_CUDA(cudaStreamWaitEvent(s, ws->ev_edge, 0));
        return ENTRO_OK;
    };
    const entro_status st = enqueue();
    // Whatever was queued, on the copy streams or the caller's, has finished with the caller's
    // buffers before the call returns, on the error paths too.
    const cudaError_t e_in = cudaStreamSynchronize(ws->copy_in), e_out = cudaStreamSynchronize(ws->copy_out),
                      e_s = cudaStreamSynchronize(s);
    if (st != ENTRO_OK) return st;
    return (e_in == cudaSuccess && e_out == cudaSuccess && e_s == cudaSuccess) ? ENTRO_OK : ENTRO_ERR_CUDA;
}

// ------------------------------------------------------------------ matrix-vector products

namespace entro {
namespace {

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

namespace entro {
namespace {

// Sizes and places of everything a fused matrix-vector call keeps on the device:
// [DevTensor x n][item_start][GemvTensor x n] (uploaded) [tables x n][fp32 sums][counts of pending parts].
struct GemvLayout {
    int n = 0;
    uint32_t lanes_batch = 1;        // accumulators per lane: the largest batch rounded up to 1, 2, 4 or 8
    uint32_t x_bytes = 0;            // shared memory for x of that many tokens
    size_t tensors_at = 0, items_at = 0, gemv_at = 0, upload_bytes = 0;
    size_t tables_at = 0, y32_at = 0, pending_at = 0, total_bytes = 0;
};

entro_status gemv_layout(const entro_tensor_desc* descs, const entro_gemv_io* io, int ntensors, GemvLayout& L)
{
    if (ntensors < 0 || (ntensors > 0 && (!descs || !io))) return ENTRO_ERR_INVALID_ARG;
    uint64_t sum_rows = 0, sum_batch_rows = 0;
    uint32_t max_batch = 1;
    for (int i = 0; i < ntensors; ++i) {
        const entro_tensor_desc& d = descs[i];
        const entro_gemv_io& g = io[i];
        if (d.n == 0) return ENTRO_ERR_INVALID_ARG;
        entro_status st = validate_desc(d, false);
        if (st != ENTRO_OK) return st;
        if (!g.x_fp16_dev || !g.y_fp16_dev || !aligned(g.x_fp16_dev, 16) || !aligned(g.y_fp16_dev, 2))
            return ENTRO_ERR_INVALID_ARG;
        if (g.rows == 0 || g.cols == 0 || (uint64_t)g.rows * g.cols != d.n) return ENTRO_ERR_INVALID_ARG;
        if (g.batch < 1 || g.batch > ENTRO_GEMV_MAX_BATCH || g.reserved != 0) return ENTRO_ERR_INVALID_ARG;
        if ((uint64_t)g.rows * g.batch > 0xffffffffull) return ENTRO_ERR_UNSUPPORTED;
        if (g.cols % 256u || (uint64_t)g.cols * g.batch > kGemvMaxX || d.chunk_symbols % 256u) return ENTRO_ERR_UNSUPPORTED;
        sum_rows += g.rows;
        sum_batch_rows += (uint64_t)g.rows * g.batch;
        if (g.batch > max_batch) max_batch = g.batch;
    }
    L.n = ntensors;
    L.lanes_batch = max_batch <= 1 ? 1u : max_batch <= 2 ? 2u : max_batch <= 4 ? 4u : 8u;
    L.x_bytes = 0;
    for (int i = 0; i < ntensors; ++i) {
        const uint32_t need = (io[i].cols * L.lanes_batch * 2u + 127u) & ~127u;
        if (need > L.x_bytes) L.x_bytes = need;
    }
    if (L.x_bytes > 2u * kGemvMaxX) return ENTRO_ERR_UNSUPPORTED;   // a wide matrix beside a larger batch elsewhere in the call
    auto up16 = [](size_t v) { return (v + 15) & ~(size_t)15; };
    size_t at = 0;
    L.tensors_at = at, at += (size_t)ntensors * sizeof(DevTensor);
    L.items_at = at, at += up16(((size_t)ntensors + 1) * 4);
    L.gemv_at = at, at += (size_t)ntensors * sizeof(GemvTensor);
    L.upload_bytes = at;
    L.tables_at = at, at += (size_t)ntensors * sizeof(TensorTables);
    L.y32_at = at, at += up16(sum_batch_rows * 4);
    L.pending_at = at, at += up16(sum_rows * 4);
    L.total_bytes = at;
    return ENTRO_OK;
}

// Fills the upload area (host copy at `host`, to live at `dev` on the device); -> number of
// work items, or 0 if there are too many.
uint64_t gemv_fill(const GemvLayout& L, const DecodeConfig& cfg, int sm_count, const entro_tensor_desc* descs,
                   const entro_gemv_io* io, char* host, char* dev)
{
    ItemPlan plan = plan_items(cfg, descs, L.n, sm_count);
    DevTensor* ht = reinterpret_cast<DevTensor*>(host + L.tensors_at);
    uint32_t* hitems = reinterpret_cast<uint32_t*>(host + L.items_at);
    GemvTensor* hg = reinterpret_cast<GemvTensor*>(host + L.gemv_at);
    float* y32 = reinterpret_cast<float*>(dev + L.y32_at);
    uint32_t* pending = reinterpret_cast<uint32_t*>(dev + L.pending_at);
    uint64_t items = 0, row0 = 0, brow0 = 0;
    for (int i = 0; i < L.n; ++i) {
        hitems[i] = (uint32_t)items;
        items += fill_dev_tensor(descs[i], plan, ht[i]);
        if (items > 0x7fffffffull) return 0;
        hg[i].x = static_cast<const uint16_t*>(io[i].x_fp16_dev);
        hg[i].y32 = y32 + brow0;
        hg[i].y = static_cast<uint16_t*>(io[i].y_fp16_dev);
        hg[i].rows = io[i].rows;
        hg[i].cols = io[i].cols;
        hg[i].batch = io[i].batch;
        hg[i].pad = 0;
        hg[i].pending = pending + row0;
        row0 += io[i].rows;
        brow0 += (uint64_t)io[i].rows * io[i].batch;
    }
    hitems[L.n] = (uint32_t)items;
    return items;
}

}  // namespace
}  // namespace entro

extern "C" entro_status entro_decode_dequant_gemv(const entro_tensor_desc* descs_host, const entro_gemv_io* io_host,
                                                  int ntensors, void* cuda_stream)
{
    GemvLayout L;
    entro_status st = gemv_layout(descs_host, io_host, ntensors, L);
    if (st != ENTRO_OK) return st;
    if (ntensors == 0) return ENTRO_OK;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    Guard guard;
    Workspace* ws = workspace();
    if (!ws) return ENTRO_ERR_CUDA;
    const DecodeConfig cfg = decode_config();
    if (!reserve_pinned(ws, L.upload_bytes)) return ENTRO_ERR_CUDA;
    if (!reserve_device(ws, L.total_bytes)) return ENTRO_ERR_CUDA;
    char* base = static_cast<char*>(ws->dev);
    const uint64_t items = gemv_fill(L, cfg, ws->sm_count, descs_host, io_host, static_cast<char*>(ws->pinned), base);
    if (items == 0) return ENTRO_ERR_UNSUPPORTED;
    DevTensor* dt = reinterpret_cast<DevTensor*>(base + L.tensors_at);
    GemvTensor* dg = reinterpret_cast<GemvTensor*>(base + L.gemv_at);
    TensorTables* dtables = reinterpret_cast<TensorTables*>(base + L.tables_at);
    ENTRO_CUDA(cudaMemcpyAsync(base, ws->pinned, L.upload_bytes, cudaMemcpyHostToDevice, s));
    mark_pinned_in_use(ws, s);
    build_tables_kernel<<<dim3((unsigned)ntensors, table_slices(ntensors, ws->sm_count)), 256, 0, s>>>(dt, cfg.lut_bits, dtables, ws->control, dg);
    count_launch();
    ENTRO_CUDA(cudaGetLastError());
    return launch_decode_any(ws, cfg, dt, ntensors, reinterpret_cast<uint32_t*>(base + L.items_at), (uint32_t)items,
                             dtables, s, dg, kSinkGemv, (int)L.lanes_batch, L.x_bytes);
}

// ------------------------------------------------------------------ prepared matrix-vector products

struct entro_gemv_plan {
    int device = -1;
    GemvLayout L;
    DecodeConfig cfg;
    char* dev = nullptr;
    uint32_t items = 0;
};

extern "C" entro_status entro_gemv_prepare(const entro_tensor_desc* descs_host, const entro_gemv_io* io_host,
                                           int ntensors, void* cuda_stream, entro_gemv_plan** plan_out)
{
    if (!plan_out) return ENTRO_ERR_INVALID_ARG;
    *plan_out = nullptr;
    if (ntensors <= 0) return ENTRO_ERR_INVALID_ARG;
    Guard guard;
    Workspace* ws = workspace();
    if (!ws) return ENTRO_ERR_CUDA;
    const DecodeConfig cfg = decode_config();
    GemvLayout L;
    entro_status st = gemv_layout(descs_host, io_host, ntensors, L);
    if (st != ENTRO_OK) return st;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    entro_gemv_plan* plan = new (std::nothrow) entro_gemv_plan;
    if (!plan) return ENTRO_ERR_CUDA;
    plan->device = ws->device;
    plan->L = L;
    plan->cfg = cfg;
    void* host = nullptr;
    auto fail = [&](entro_status why) {
        if (host) cudaFreeHost(host);
        if (plan->dev) cudaFree(plan->dev);
        delete plan;
        return why;
    };
    if (cudaMalloc(reinterpret_cast<void**>(&plan->dev), L.total_bytes) != cudaSuccess) return fail(ENTRO_ERR_CUDA);
    if (cudaMallocHost(&host, L.upload_bytes) != cudaSuccess) return fail(ENTRO_ERR_CUDA);
    const uint64_t items = gemv_fill(L, cfg, ws->sm_count, descs_host, io_host, static_cast<char*>(host), plan->dev);
    if (items == 0) return fail(ENTRO_ERR_UNSUPPORTED);
    plan->items = (uint32_t)items;
    if (cudaMemcpyAsync(plan->dev, host, L.upload_bytes, cudaMemcpyHostToDevice, s) != cudaSuccess) return fail(ENTRO_ERR_CUDA);
    build_tables_kernel<<<dim3((unsigned)ntensors, table_slices(ntensors, ws->sm_count)), 256, 0, s>>>(
        reinterpret_cast<DevTensor*>(plan->dev + L.tensors_at), cfg.lut_bits,
        reinterpret_cast<TensorTables*>(plan->dev + L.tables_at), ws->control,
        reinterpret_cast<GemvTensor*>(plan->dev + L.gemv_at));
    count_launch();
    if (cudaGetLastError() != cudaSuccess || cudaStreamSynchronize(s) != cudaSuccess) return fail(ENTRO_ERR_CUDA);
    cudaFreeHost(host);
    *plan_out = plan;
    return ENTRO_OK;
}

extern "C" entro_status entro_gemv_run(entro_gemv_plan* plan, void* cuda_stream)
{
    if (!plan || !plan->dev) return ENTRO_ERR_INVALID_ARG;
    Guard guard;
    Workspace* ws = workspace();
    if (!ws) return ENTRO_ERR_CUDA;
    if (ws->device != plan->device) return ENTRO_ERR_INVALID_ARG;
    const GemvLayout& L = plan->L;
    return launch_decode_any(ws, plan->cfg, reinterpret_cast<DevTensor*>(plan->dev + L.tensors_at), L.n,
                             reinterpret_cast<uint32_t*>(plan->dev + L.items_at), plan->items,
                             reinterpret_cast<TensorTables*>(plan->dev + L.tables_at), (cudaStream_t)cuda_stream,
                             reinterpret_cast<GemvTensor*>(plan->dev + L.gemv_at), kSinkGemv, (int)L.lanes_batch,
                             L.x_bytes);
}

extern "C" entro_status entro_gemv_release(entro_gemv_plan* plan)
{
    if (!plan) return ENTRO_OK;
    Guard guard;
    entro_status st = ENTRO_OK;
    if (plan->dev && cudaFree(plan->dev) != cudaSuccess) st = ENTRO_ERR_CUDA;   // waits for kernels that still use it
    delete plan;
    return st;
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
    const DecodeConfig cfg = config_for(decode_config(), descs_host, ntensors, sd->max_smem_optin);   // host arithmetic only
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
    build_tables_kernel<<<dim3((unsigned)live, table_slices(live, sd->sm_count)), 256, 0, s>>>(sc->tensors, cfg.lut_bits, sc->tables, sc->control, nullptr);
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

extern "C" int entro_checked_build(void)
{
#ifdef ENTRO_CHECKED
    return 1;
#else
    return 0;
#endif
}

extern "C" long long entro_check_violations(void)
{
#ifdef ENTRO_CHECKED
    Guard g;
    unsigned int count = 0, zero = 0;
    if (cudaDeviceSynchronize() != cudaSuccess) return -1;
    if (cudaMemcpyFromSymbol(&count, g_check_violations, sizeof(count)) != cudaSuccess) return -1;
    if (cudaMemcpyToSymbol(g_check_violations, &zero, sizeof(zero)) != cudaSuccess) return -1;
    return (long long)count;
#else
    return 0;
#endif
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
