// entro_quantize_tensor and entro_histogram: the offline side of the pipeline (Section 3,
// "Mixed Quantization Scheme", Eq. 1; symbol frequencies for the Huffman tree).
#include <cuda_fp16.h>

#include <cmath>

#include "entro_internal.h"

namespace entro {
namespace {

constexpr int kThreads = 256;

struct Range {
    float lo, hi;
    uint32_t nonfinite;
    uint32_t pad;
};

__device__ __forceinline__ void scan_half(uint16_t h, float& lo, float& hi, uint32_t& bad)
{
    if ((h & 0x7c00u) == 0x7c00u) bad = 1;
    float x = __half2float(__ushort_as_half(h));
    lo = fminf(lo, x);
    hi = fmaxf(hi, x);
}

// Pass 1: per-block minimum / maximum and a non-finite flag.
__global__ void __launch_bounds__(kThreads) range_partial_kernel(const uint16_t* __restrict__ w, uint64_t n,
                                                                 Range* __restrict__ partial)
{
    float lo = INFINITY, hi = -INFINITY;
    uint32_t bad = 0;
    const uint64_t nvec = n / 8;
    const uint4* wv = reinterpret_cast<const uint4*>(w);
    for (uint64_t i = blockIdx.x * (uint64_t)kThreads + threadIdx.x; i < nvec; i += (uint64_t)gridDim.x * kThreads) {
        uint4 v = __ldg(wv + i);
        uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            scan_half((uint16_t)(u[k] & 0xffffu), lo, hi, bad);
            scan_half((uint16_t)(u[k] >> 16), lo, hi, bad);
        }
    }
    if (blockIdx.x == 0) {
        for (uint64_t i = nvec * 8 + threadIdx.x; i < n; i += kThreads) scan_half(w[i], lo, hi, bad);
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, d));
        hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, d));
        bad |= __shfl_xor_sync(0xffffffffu, bad, d);
    }
    __shared__ Range s[kThreads / 32];
    if ((threadIdx.x & 31) == 0) s[threadIdx.x >> 5] = {lo, hi, bad, 0};
    __syncthreads();
    if (threadIdx.x == 0) {
        Range r = s[0];
        for (int k = 1; k < kThreads / 32; ++k) {
            r.lo = fminf(r.lo, s[k].lo);
            r.hi = fmaxf(r.hi, s[k].hi);
            r.nonfinite |= s[k].nonfinite;
        }
        partial[blockIdx.x] = r;
    }
}

// Pass 2: one block folds the partials.
__global__ void __launch_bounds__(kThreads) range_final_kernel(const Range* __restrict__ partial, int count,
                                                               Range* __restrict__ result)
{
    float lo = INFINITY, hi = -INFINITY;
    uint32_t bad = 0;
    for (int i = threadIdx.x; i < count; i += kThreads) {
        lo = fminf(lo, partial[i].lo);
        hi = fmaxf(hi, partial[i].hi);
        bad |= partial[i].nonfinite;
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, d));
        hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, d));
        bad |= __shfl_xor_sync(0xffffffffu, bad, d);
    }
    __shared__ Range s[kThreads / 32];
    if ((threadIdx.x & 31) == 0) s[threadIdx.x >> 5] = {lo, hi, bad, 0};
    __syncthreads();
    if (threadIdx.x == 0) {
        Range r = s[0];
        for (int k = 1; k < kThreads / 32; ++k) {
            r.lo = fminf(r.lo, s[k].lo);
            r.hi = fmaxf(r.hi, s[k].hi);
            r.nonfinite |= s[k].nonfinite;
        }
        *result = r;
    }
}

// q = clamp(rne(w / s) + z, 0, qmax): IEEE division, round-half-to-even conversion.
__device__ __forceinline__ uint32_t quantise_one(uint16_t h, float s, int z, int qmax)
{
    float x = __half2float(__ushort_as_half(h));
    int q = __float2int_rn(__fdiv_rn(x, s)) + z;
    return (uint32_t)min(max(q, 0), qmax);
}

__global__ void __launch_bounds__(kThreads) quantise_kernel(const uint16_t* __restrict__ w, uint64_t n, float s,
                                                            int z, int qmax, uint8_t* __restrict__ q)
{
    const uint64_t nvec = n / 8;
    const uint4* wv = reinterpret_cast<const uint4*>(w);
    uint2* qv = reinterpret_cast<uint2*>(q);
    for (uint64_t i = blockIdx.x * (uint64_t)kThreads + threadIdx.x; i < nvec; i += (uint64_t)gridDim.x * kThreads) {
        uint4 v = __ldg(wv + i);
        uint32_t u[4] = {v.x, v.y, v.z, v.w};
        uint32_t b[8];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            b[2 * k] = quantise_one((uint16_t)(u[k] & 0xffffu), s, z, qmax);
            b[2 * k + 1] = quantise_one((uint16_t)(u[k] >> 16), s, z, qmax);
        }
        uint2 o;
        o.x = b[0] | (b[1] << 8) | (b[2] << 16) | (b[3] << 24);
        o.y = b[4] | (b[5] << 8) | (b[6] << 16) | (b[7] << 24);
        qv[i] = o;
    }
    if (blockIdx.x == 0) {
        for (uint64_t i = nvec * 8 + threadIdx.x; i < n; i += kThreads) q[i] = (uint8_t)quantise_one(w[i], s, z, qmax);
    }
}

// (s, z) of one tensor on the device, by the arithmetic of the host code in
// entro_quantize_tensor (IEEE fp32, one rounding per operation), so that a batch of tensors
// needs no round trip to the host between the range pass and the quantise pass.
struct DevQParams {
    float scale;
    int32_t zero_point;
    int32_t mode;
    uint32_t nonfinite;
    float lo, hi;
    uint32_t pad[2];
};

__device__ __forceinline__ void derive_params(const Range* range, int qmax, int mode, DevQParams* out)
{
    float lo = range->lo, hi = range->hi;
    if (lo == 0.0f) lo = 0.0f;   // -0 and +0 are the same bound
    if (hi == 0.0f) hi = 0.0f;
    int resolved = mode;
    if (resolved == ENTRO_MODE_AUTO) resolved = (lo >= 0.0f) ? ENTRO_MODE_UNSIGNED : ENTRO_MODE_ASYMMETRIC;
    float s;
    int z = 0;
    if (resolved == ENTRO_MODE_UNSIGNED) {
        s = __fdiv_rn(hi, (float)qmax);
        if (!(s > 0.0f)) s = 1.0f;
    } else {
        s = __fdiv_rn(__fsub_rn(hi, lo), (float)qmax);
        if (!(s > 0.0f)) s = 1.0f;
        float zr = rintf(__fdiv_rn(-lo, s));
        zr = zr < 0.0f ? 0.0f : (zr > (float)qmax ? (float)qmax : zr);
        z = (int)zr;
    }
    out->scale = s;
    out->zero_point = z;
    out->mode = resolved;
    out->nonfinite = range->nonfinite;
    out->lo = lo;
    out->hi = hi;
    out->pad[0] = out->pad[1] = 0;
}

// Pass 2 of a batch: fold the partials, then derive the parameters in the same launch.
__global__ void __launch_bounds__(kThreads) range_final_params_kernel(const Range* __restrict__ partial, int count,
                                                                      int qmax, int mode, DevQParams* __restrict__ out)
{
    float lo = INFINITY, hi = -INFINITY;
    uint32_t bad = 0;
    for (int i = threadIdx.x; i < count; i += kThreads) {
        lo = fminf(lo, partial[i].lo);
        hi = fmaxf(hi, partial[i].hi);
        bad |= partial[i].nonfinite;
    }
#pragma unroll
    for (int d = 16; d > 0; d >>= 1) {
        lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, d));
        hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, d));
        bad |= __shfl_xor_sync(0xffffffffu, bad, d);
    }
    __shared__ Range s[kThreads / 32];
    if ((threadIdx.x & 31) == 0) s[threadIdx.x >> 5] = {lo, hi, bad, 0};
    __syncthreads();
    if (threadIdx.x == 0) {
        Range r = s[0];
        for (int k = 1; k < kThreads / 32; ++k) {
            r.lo = fminf(r.lo, s[k].lo);
            r.hi = fmaxf(r.hi, s[k].hi);
            r.nonfinite |= s[k].nonfinite;
        }
        derive_params(&r, qmax, mode, out);
    }
}

// Quantise and count in one pass over the weights: q as quantise_kernel writes it, counts as
// histogram_kernel counts them.  Nothing is written for a tensor that holds a NaN or an infinity.
__global__ void __launch_bounds__(kThreads) quantise_count_kernel(const uint16_t* __restrict__ w, uint64_t n,
                                                                  const DevQParams* __restrict__ p, int qmax,
                                                                  uint8_t* __restrict__ q,
                                                                  unsigned long long* __restrict__ counts)
{
    if (p->nonfinite) return;
    __shared__ uint32_t hist[kThreads / 32][ENTRO_MAX_SYMBOLS];
    for (int i = threadIdx.x; i < (kThreads / 32) * ENTRO_MAX_SYMBOLS; i += kThreads) (&hist[0][0])[i] = 0;
    __syncthreads();
    uint32_t* mine = hist[threadIdx.x >> 5];
    const float s = p->scale;
    const int z = p->zero_point;
    const uint64_t nvec = n / 8;
    const uint4* wv = reinterpret_cast<const uint4*>(w);
    uint2* qv = reinterpret_cast<uint2*>(q);
    for (uint64_t i = blockIdx.x * (uint64_t)kThreads + threadIdx.x; i < nvec; i += (uint64_t)gridDim.x * kThreads) {
        uint4 v = __ldg(wv + i);
        uint32_t u[4] = {v.x, v.y, v.z, v.w};
        uint32_t b[8];
#pragma unroll
        for (int k = 0; k < 4; ++k) {
            b[2 * k] = quantise_one((uint16_t)(u[k] & 0xffffu), s, z, qmax);
            b[2 * k + 1] = quantise_one((uint16_t)(u[k] >> 16), s, z, qmax);
        }
#pragma unroll
        for (int k = 0; k < 8; ++k) atomicAdd(&mine[b[k]], 1u);
        uint2 o;
        o.x = b[0] | (b[1] << 8) | (b[2] << 16) | (b[3] << 24);
        o.y = b[4] | (b[5] << 8) | (b[6] << 16) | (b[7] << 24);
        qv[i] = o;
    }
    if (blockIdx.x == 0) {
        for (uint64_t i = nvec * 8 + threadIdx.x; i < n; i += kThreads) {
            const uint32_t sym = quantise_one(w[i], s, z, qmax);
            q[i] = (uint8_t)sym;
            atomicAdd(&mine[sym], 1u);
        }
    }
    __syncthreads();
    for (uint32_t k = threadIdx.x; k <= (uint32_t)qmax; k += kThreads) {
        unsigned long long t = 0;
        for (int wi = 0; wi < kThreads / 32; ++wi) t += hist[wi][k];
        if (t) atomicAdd(&counts[k], t);
    }
}

// Block-based grid: one warp per block of `block` consecutive weights.  The warp finds the
// block's range, every lane derives the same (s, z) from it with the arithmetic of the
// per-tensor call (IEEE fp32, one rounding per operation), then the block is quantised.
__global__ void __launch_bounds__(kThreads) quantise_blocks_kernel(const uint16_t* __restrict__ w, uint64_t n,
                                                                   uint32_t block, uint64_t nblocks, int qmax, int mode,
                                                                   uint8_t* __restrict__ q, float* __restrict__ scales,
                                                                   int32_t* __restrict__ zps,
                                                                   uint32_t* __restrict__ nonfinite)
{
    const uint32_t lane = threadIdx.x & 31u;
    const uint64_t warps = ((uint64_t)gridDim.x * kThreads) >> 5;
    for (uint64_t b = ((uint64_t)blockIdx.x * kThreads + threadIdx.x) >> 5; b < nblocks; b += warps) {
        const uint64_t first = b * block;
        const uint32_t m = (uint32_t)min((uint64_t)block, n - first);
        float lo = INFINITY, hi = -INFINITY;
        uint32_t bad = 0;
        for (uint32_t i = lane; i < m; i += 32u) scan_half(w[first + i], lo, hi, bad);
#pragma unroll
        for (int d = 16; d > 0; d >>= 1) {
            lo = fminf(lo, __shfl_xor_sync(0xffffffffu, lo, d));
            hi = fmaxf(hi, __shfl_xor_sync(0xffffffffu, hi, d));
            bad |= __shfl_xor_sync(0xffffffffu, bad, d);
        }
        if (bad) {
            if (lane == 0) atomicOr(nonfinite, 1u);
            continue;
        }
        if (lo == 0.0f) lo = 0.0f;   // -0 and +0 are the same bound
        if (hi == 0.0f) hi = 0.0f;
        const bool unsigned_grid = mode == ENTRO_MODE_UNSIGNED || (mode == ENTRO_MODE_AUTO && lo >= 0.0f);
        float s;
        int z = 0;
        if (unsigned_grid) {
            s = __fdiv_rn(hi, (float)qmax);
            if (!(s > 0.0f)) s = 1.0f;
        } else {
            s = __fdiv_rn(__fsub_rn(hi, lo), (float)qmax);
            if (!(s > 0.0f)) s = 1.0f;
            float zr = rintf(__fdiv_rn(-lo, s));
            zr = zr < 0.0f ? 0.0f : (zr > (float)qmax ? (float)qmax : zr);
            z = (int)zr;
        }
        for (uint32_t i = lane; i < m; i += 32u) q[first + i] = (uint8_t)quantise_one(w[first + i], s, z, qmax);
        if (lane == 0) {
            if (scales) scales[b] = s;
            if (zps) zps[b] = z;
        }
    }
}

// Per-warp shared-memory histograms, merged into 64-bit global counters.
__global__ void __launch_bounds__(kThreads) histogram_kernel(const uint8_t* __restrict__ q, uint64_t n, uint32_t nsym,
                                                             unsigned long long* __restrict__ counts,
                                                             uint32_t* __restrict__ bad_symbol)
{
    __shared__ uint32_t hist[kThreads / 32][ENTRO_MAX_SYMBOLS];
    for (int i = threadIdx.x; i < (kThreads / 32) * ENTRO_MAX_SYMBOLS; i += kThreads) (&hist[0][0])[i] = 0;
    __syncthreads();
    uint32_t* mine = hist[threadIdx.x >> 5];
    uint32_t bad = 0;
    const uint64_t nvec = n / 16;
    const uint4* qv = reinterpret_cast<const uint4*>(q);
    // Each block handles a bounded slice so the 32-bit shared counters cannot overflow.
    for (uint64_t i = blockIdx.x * (uint64_t)kThreads + threadIdx.x; i < nvec; i += (uint64_t)gridDim.x * kThreads) {
        uint4 v = __ldg(qv + i);
        uint32_t u[4] = {v.x, v.y, v.z, v.w};
#pragma unroll
        for (int k = 0; k < 4; ++k) {
#pragma unroll
            for (int b = 0; b < 4; ++b) {
                uint32_t sym = (u[k] >> (8 * b)) & 0xffu;
                if (sym < nsym) atomicAdd(&mine[sym], 1u);
                else bad = 1;
            }
        }
    }
    if (blockIdx.x == 0) {
        for (uint64_t i = nvec * 16 + threadIdx.x; i < n; i += kThreads) {
            uint32_t sym = q[i];
            if (sym < nsym) atomicAdd(&mine[sym], 1u);
            else bad = 1;
        }
    }
    if (bad) atomicOr(bad_symbol, 1u);
    __syncthreads();
    for (uint32_t k = threadIdx.x; k < nsym; k += kThreads) {
        unsigned long long t = 0;
        for (int wi = 0; wi < kThreads / 32; ++wi) t += hist[wi][k];
        if (t) atomicAdd(&counts[k], t);
    }
}

int grid_for(uint64_t work_items, int sm_count, int per_sm)
{
    uint64_t blocks = (work_items + kThreads - 1) / kThreads;
    uint64_t cap = (uint64_t)sm_count * per_sm;
    if (blocks < 1) blocks = 1;
    return (int)(blocks < cap ? blocks : cap);
}

}  // namespace
}  // namespace entro

using namespace entro;

extern "C" entro_status entro_quantize_tensor(const void* w_fp16_dev, uint64_t n, int bits, entro_mode mode,
                                              uint8_t* q_dev, entro_qparams* qp, void* cuda_stream)
{
    if (!w_fp16_dev || !q_dev || !qp || n == 0 || (bits != 4 && bits != 8)) return ENTRO_ERR_INVALID_ARG;
    if (mode != ENTRO_MODE_AUTO && mode != ENTRO_MODE_UNSIGNED && mode != ENTRO_MODE_ASYMMETRIC)
        return ENTRO_ERR_INVALID_ARG;
    if (!aligned(w_fp16_dev, 16) || !aligned(q_dev, 16)) return ENTRO_ERR_INVALID_ARG;
    Guard g;
    Workspace* ws = workspace();
    if (!ws) return ENTRO_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const uint16_t* w = static_cast<const uint16_t*>(w_fp16_dev);

    int grid = grid_for(n / 8 + 1, ws->sm_count, 8);
    if (!reserve_device(ws, (size_t)(grid + 1) * sizeof(Range))) return ENTRO_ERR_CUDA;
    if (!reserve_pinned(ws, sizeof(Range))) return ENTRO_ERR_CUDA;
    Range* partial = static_cast<Range*>(ws->dev);
    Range* result = partial + grid;
    range_partial_kernel<<<grid, kThreads, 0, s>>>(w, n, partial);
    range_final_kernel<<<1, kThreads, 0, s>>>(partial, grid, result);
    count_launch(2);
    ENTRO_CUDA(cudaGetLastError());
    Range* host = static_cast<Range*>(ws->pinned);
    ENTRO_CUDA(cudaMemcpyAsync(host, result, sizeof(Range), cudaMemcpyDeviceToHost, s));
    ENTRO_CUDA(cudaStreamSynchronize(s));
    if (host->nonfinite) return ENTRO_ERR_NONFINITE;

    // (s, z) from the range, in fp32, one rounding per operation.
    float lo = host->lo, hi = host->hi;
    if (lo == 0.0f) lo = 0.0f;   // -0 and +0 are the same bound
    if (hi == 0.0f) hi = 0.0f;
    const int qmax = (1 << bits) - 1;
    int resolved = mode;
    if (resolved == ENTRO_MODE_AUTO) resolved = (lo >= 0.0f) ? ENTRO_MODE_UNSIGNED : ENTRO_MODE_ASYMMETRIC;
    volatile float scale;
    int zp = 0;
    if (resolved == ENTRO_MODE_UNSIGNED) {
        scale = hi / (float)qmax;
        if (!(scale > 0.0f)) scale = 1.0f;
    } else {
        volatile float range = hi - lo;
        scale = range / (float)qmax;
        if (!(scale > 0.0f)) scale = 1.0f;
        volatile float zf = -lo / scale;
        float zr = std::nearbyintf(zf);
        zr = zr < 0.0f ? 0.0f : (zr > (float)qmax ? (float)qmax : zr);
        zp = (int)zr;
    }
    qp->bits = bits;
    qp->mode = resolved;
    qp->scale = scale;
    qp->zero_point = zp;
    qp->lo = lo;
    qp->hi = hi;

    quantise_kernel<<<grid_for(n / 8 + 1, ws->sm_count, 8), kThreads, 0, s>>>(w, n, scale, zp, qmax, q_dev);
    count_launch();
    ENTRO_CUDA(cudaGetLastError());
    ENTRO_CUDA(cudaStreamSynchronize(s));
    return ENTRO_OK;
}

extern "C" entro_status entro_quantize_histogram_batched(const entro_quantize_job* jobs, int njobs,
                                                         entro_qparams* qp_host, uint64_t* counts_host,
                                                         void* cuda_stream)
{
    if (njobs < 0 || (njobs > 0 && (!jobs || !qp_host || !counts_host))) return ENTRO_ERR_INVALID_ARG;
    if (njobs == 0) return ENTRO_OK;
    for (int j = 0; j < njobs; ++j) {
        const entro_quantize_job& job = jobs[j];
        if (!job.w_fp16_dev || !job.q_dev || job.n == 0 || (job.bits != 4 && job.bits != 8)) return ENTRO_ERR_INVALID_ARG;
        if (job.mode != ENTRO_MODE_AUTO && job.mode != ENTRO_MODE_UNSIGNED && job.mode != ENTRO_MODE_ASYMMETRIC)
            return ENTRO_ERR_INVALID_ARG;
        if (!aligned(job.w_fp16_dev, 16) || !aligned(job.q_dev, 16)) return ENTRO_ERR_INVALID_ARG;
    }
    Guard g;
    Workspace* ws = workspace();
    if (!ws) return ENTRO_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    // device area: [partial ranges of the tensor in flight][parameters x njobs][counts x njobs x 256]
    const int max_grid = ws->sm_count * 8;
    const size_t partial_bytes = (size_t)max_grid * sizeof(Range);
    const size_t params_bytes = (size_t)njobs * sizeof(DevQParams);
    const size_t counts_bytes = (size_t)njobs * ENTRO_MAX_SYMBOLS * sizeof(unsigned long long);
    if (!reserve_device(ws, partial_bytes + params_bytes + counts_bytes)) return ENTRO_ERR_CUDA;
    if (!reserve_pinned(ws, params_bytes + counts_bytes)) return ENTRO_ERR_CUDA;
    char* base = static_cast<char*>(ws->dev);
    Range* partial = reinterpret_cast<Range*>(base);
    DevQParams* params = reinterpret_cast<DevQParams*>(base + partial_bytes);
    unsigned long long* counts = reinterpret_cast<unsigned long long*>(base + partial_bytes + params_bytes);
    ENTRO_CUDA(cudaMemsetAsync(counts, 0, counts_bytes, s));
    for (int j = 0; j < njobs; ++j) {
        const entro_quantize_job& job = jobs[j];
        const uint16_t* w = static_cast<const uint16_t*>(job.w_fp16_dev);
        const int qmax = (1 << job.bits) - 1;
        int grid = grid_for(job.n / 8 + 1, ws->sm_count, 8);
        // at most 2^31 symbols per block keeps the 32-bit shared counters exact
        if ((uint64_t)grid < (job.n >> 31) + 1) grid = (int)((job.n >> 31) + 1);
        if (grid > max_grid) return ENTRO_ERR_UNSUPPORTED;
        range_partial_kernel<<<grid, kThreads, 0, s>>>(w, job.n, partial);
        range_final_params_kernel<<<1, kThreads, 0, s>>>(partial, grid, qmax, job.mode, params + j);
        quantise_count_kernel<<<grid, kThreads, 0, s>>>(w, job.n, params + j, qmax, job.q_dev,
                                                        counts + (size_t)j * ENTRO_MAX_SYMBOLS);
        count_launch(3);
    }
    ENTRO_CUDA(cudaGetLastError());
    char* host = static_cast<char*>(ws->pinned);
    ENTRO_CUDA(cudaMemcpyAsync(host, params, params_bytes + counts_bytes, cudaMemcpyDeviceToHost, s));
    ENTRO_CUDA(cudaStreamSynchronize(s));
    const DevQParams* hp = reinterpret_cast<const DevQParams*>(host);
    const unsigned long long* hc = reinterpret_cast<const unsigned long long*>(host + params_bytes);
    entro_status st = ENTRO_OK;
    for (int j = 0; j < njobs; ++j) {
        qp_host[j].bits = jobs[j].bits;
        qp_host[j].mode = hp[j].mode;
        qp_host[j].scale = hp[j].scale;
        qp_host[j].zero_point = hp[j].zero_point;
        qp_host[j].lo = hp[j].lo;
        qp_host[j].hi = hp[j].hi;
        for (int k = 0; k < ENTRO_MAX_SYMBOLS; ++k) counts_host[(size_t)j * ENTRO_MAX_SYMBOLS + k] = hc[(size_t)j * ENTRO_MAX_SYMBOLS + k];
        if (hp[j].nonfinite) st = ENTRO_ERR_NONFINITE;
    }
    return st;
}

extern "C" entro_status entro_quantize_blocks(const void* w_fp16_dev, uint64_t n, int bits, entro_mode mode,
                                              uint32_t block, uint8_t* q_dev, float* scales_dev,
                                              int32_t* zero_points_dev, void* cuda_stream)
{
    if (!w_fp16_dev || !q_dev || n == 0 || block == 0 || (bits != 4 && bits != 8)) return ENTRO_ERR_INVALID_ARG;
    if (mode != ENTRO_MODE_AUTO && mode != ENTRO_MODE_UNSIGNED && mode != ENTRO_MODE_ASYMMETRIC)
        return ENTRO_ERR_INVALID_ARG;
    if (!aligned(w_fp16_dev, 2) || (scales_dev && !aligned(scales_dev, 4)) || (zero_points_dev && !aligned(zero_points_dev, 4)))
        return ENTRO_ERR_INVALID_ARG;
    Guard g;
    Workspace* ws = workspace();
    if (!ws) return ENTRO_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    if (!reserve_device(ws, 16) || !reserve_pinned(ws, 16)) return ENTRO_ERR_CUDA;
    uint32_t* flag = static_cast<uint32_t*>(ws->dev);
    ENTRO_CUDA(cudaMemsetAsync(flag, 0, 4, s));
    const uint64_t nblocks = (n + block - 1) / block;
    const int grid = grid_for(nblocks * 32, ws->sm_count, 8);
    quantise_blocks_kernel<<<grid, kThreads, 0, s>>>(static_cast<const uint16_t*>(w_fp16_dev), n, block, nblocks,
                                                     (1 << bits) - 1, (int)mode, q_dev, scales_dev, zero_points_dev, flag);
    count_launch();
    ENTRO_CUDA(cudaGetLastError());
    uint32_t* host = static_cast<uint32_t*>(ws->pinned);
    ENTRO_CUDA(cudaMemcpyAsync(host, flag, 4, cudaMemcpyDeviceToHost, s));
    ENTRO_CUDA(cudaStreamSynchronize(s));
    return *host ? ENTRO_ERR_NONFINITE : ENTRO_OK;
}

extern "C" entro_status entro_histogram(const uint8_t* q_dev, uint64_t n, int bits, uint64_t* counts_host,
                                        void* cuda_stream)
{
    if (!q_dev || !counts_host || (bits != 4 && bits != 8)) return ENTRO_ERR_INVALID_ARG;
    if (!aligned(q_dev, 16)) return ENTRO_ERR_INVALID_ARG;
    const uint32_t nsym = 1u << bits;
    Guard g;
    Workspace* ws = workspace();
    if (!ws) return ENTRO_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    const size_t bytes = (ENTRO_MAX_SYMBOLS + 1) * sizeof(unsigned long long);
    if (!reserve_device(ws, bytes) || !reserve_pinned(ws, bytes)) return ENTRO_ERR_CUDA;
    unsigned long long* counts = static_cast<unsigned long long*>(ws->dev);
    uint32_t* bad = reinterpret_cast<uint32_t*>(counts + ENTRO_MAX_SYMBOLS);
    ENTRO_CUDA(cudaMemsetAsync(counts, 0, bytes, s));
    if (n) {
        // At most 2^31 symbols per block keeps the 32-bit shared counters exact.
        uint64_t min_blocks = (n >> 31) + 1;
        int grid = grid_for(n / 16 + 1, ws->sm_count, 8);
        if ((uint64_t)grid < min_blocks) grid = (int)min_blocks;
        histogram_kernel<<<grid, kThreads, 0, s>>>(q_dev, n, nsym, counts, bad);
        count_launch();
        ENTRO_CUDA(cudaGetLastError());
    }
    unsigned long long* host = static_cast<unsigned long long*>(ws->pinned);
    ENTRO_CUDA(cudaMemcpyAsync(host, counts, bytes, cudaMemcpyDeviceToHost, s));
    ENTRO_CUDA(cudaStreamSynchronize(s));
    if (*reinterpret_cast<uint32_t*>(host + ENTRO_MAX_SYMBOLS)) return ENTRO_ERR_INVALID_ARG;
    for (uint32_t k = 0; k < nsym; ++k) counts_host[k] = host[k];
    return ENTRO_OK;
}
