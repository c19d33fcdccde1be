// Per-device workspace, status word and small utility entry points.
#include <atomic>
#include <mutex>

#include "entro_internal.h"

namespace entro {

namespace {
constexpr int kMaxDevices = 64;
Workspace g_ws[kMaxDevices];
std::mutex g_mutex;
std::atomic<uint64_t> g_launches{0};
DecodeConfig g_cfg;
}  // namespace

void lock() { g_mutex.lock(); }
void unlock() { g_mutex.unlock(); }
void count_launch(int n) { g_launches.fetch_add((uint64_t)n, std::memory_order_relaxed); }
DecodeConfig& decode_config() { return g_cfg; }

Workspace* workspace()
{
    int dev = -1;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= kMaxDevices) return nullptr;
    Workspace* ws = &g_ws[dev];
    if (ws->device == dev) return ws;
    cudaDeviceProp prop;
    if (cudaGetDeviceProperties(&prop, dev) != cudaSuccess) return nullptr;
    ws->sm_count = prop.multiProcessorCount;
    ws->max_smem_optin = (int)prop.sharedMemPerBlockOptin;
    if (cudaMalloc(&ws->control, 256) != cudaSuccess) return nullptr;
    if (cudaMemset(ws->control, 0, 256) != cudaSuccess) return nullptr;
    if (cudaEventCreateWithFlags(&ws->upload_done, cudaEventDisableTiming) != cudaSuccess) return nullptr;
    ws->device = dev;
    return ws;
}

bool reserve_device(Workspace* ws, size_t bytes)
{
    ws->kept = false;      // the caller is about to overwrite the area
    if (bytes <= ws->dev_bytes) return true;
    if (ws->dev) {
        // cudaFree waits for work that may still use the old area.
        if (cudaFree(ws->dev) != cudaSuccess) return false;
        ws->dev = nullptr;
        ws->dev_bytes = 0;
    }
    size_t want = bytes + bytes / 4 + 4096;
    if (cudaMalloc(&ws->dev, want) != cudaSuccess) return false;
    ws->dev_bytes = want;
    return true;
}

bool wait_pinned_free(Workspace* ws)
{
    if (!ws->upload_pending) return true;
    if (cudaEventSynchronize(ws->upload_done) != cudaSuccess) return false;
    ws->upload_pending = false;
    return true;
}

bool reserve_pinned(Workspace* ws, size_t bytes)
{
    if (!wait_pinned_free(ws)) return false;
    if (bytes <= ws->pinned_bytes) return true;
    if (ws->pinned) {
        if (cudaFreeHost(ws->pinned) != cudaSuccess) return false;
        ws->pinned = nullptr;
        ws->pinned_bytes = 0;
    }
    size_t want = bytes + bytes / 4 + 4096;
    if (cudaMallocHost(&ws->pinned, want) != cudaSuccess) return false;
    ws->pinned_bytes = want;
    return true;
}

void mark_pinned_in_use(Workspace* ws, cudaStream_t s)
{
    if (cudaEventRecord(ws->upload_done, s) == cudaSuccess) ws->upload_pending = true;
}

bool codebook_lengths_valid(const entro_codebook* cb)
{
    if (!cb || cb->nsym < 1 || cb->nsym > ENTRO_MAX_SYMBOLS) return false;
    // Kraft sum in units of 2^-32: exactly 2^32 for a complete code, 2^31 for the
    // one-symbol code; anything above 2^32 is not a prefix code.
    unsigned long long kraft = 0;
    int used = 0;
    for (int k = 0; k < cb->nsym; ++k) {
        int l = cb->len[k];
        if (l > ENTRO_MAX_CODE_LEN) return false;
        if (l) {
            kraft += 1ull << (32 - l);
            used++;
        }
    }
    for (int k = cb->nsym; k < ENTRO_MAX_SYMBOLS; ++k)
        if (cb->len[k]) return false;
    if (used == 0) return false;
    if (used == 1) return kraft == (1ull << 31);
    return kraft == (1ull << 32);
}

}  // namespace entro

using namespace entro;

extern "C" entro_status entro_last_device_status(void* cuda_stream)
{
    Guard g;
    Workspace* ws = workspace();
    if (!ws) return ENTRO_ERR_CUDA;
    cudaStream_t s = (cudaStream_t)cuda_stream;
    uint32_t st = 0;
    ENTRO_CUDA(cudaStreamSynchronize(s));
    ENTRO_CUDA(cudaMemcpyAsync(&st, ws->control + 1, sizeof(st), cudaMemcpyDeviceToHost, s));
    ENTRO_CUDA(cudaMemsetAsync(ws->control + 1, 0, sizeof(uint32_t), s));
    ENTRO_CUDA(cudaStreamSynchronize(s));
    if (st & kStatInternal) return ENTRO_ERR_UNSUPPORTED;   // the device does not lay out shared memory as the kernel expects
    return st ? ENTRO_ERR_CORRUPT_STREAM : ENTRO_OK;
}

extern "C" entro_status entro_profile_begin(int max_records)
{
    if (max_records < 0 || max_records > 65536) return ENTRO_ERR_INVALID_ARG;
    Guard g;
    Workspace* ws = workspace();
    if (!ws) return ENTRO_ERR_CUDA;
    for (int i = 0; i < ws->prof_cap; ++i) {
        cudaEventDestroy(ws->prof_start[i]);
        cudaEventDestroy(ws->prof_stop[i]);
    }
    delete[] ws->prof_start;
    delete[] ws->prof_stop;
    ws->prof_start = ws->prof_stop = nullptr;
    ws->prof_cap = ws->prof_used = 0;
    if (max_records == 0) return ENTRO_OK;
    ws->prof_start = new cudaEvent_t[max_records];
    ws->prof_stop = new cudaEvent_t[max_records];
    for (int i = 0; i < max_records; ++i) {
        ENTRO_CUDA(cudaEventCreate(&ws->prof_start[i]));
        ENTRO_CUDA(cudaEventCreate(&ws->prof_stop[i]));
        ws->prof_cap = i + 1;
    }
    return ENTRO_OK;
}

extern "C" int entro_profile_read(float* ms_host, int cap)
{
    Guard g;
    Workspace* ws = workspace();
    if (!ws || !ms_host || cap < 0) return -1;
    int n = ws->prof_used < cap ? ws->prof_used : cap;
    for (int i = 0; i < n; ++i) {
        if (cudaEventSynchronize(ws->prof_stop[i]) != cudaSuccess) return -1;
        if (cudaEventElapsedTime(&ms_host[i], ws->prof_start[i], ws->prof_stop[i]) != cudaSuccess) return -1;
    }
    ws->prof_used = 0;
    return n;
}

extern "C" uint64_t entro_kernel_launch_count(void) { return g_launches.load(); }

extern "C" const char* entro_status_string(entro_status st)
{
    switch (st) {
        case ENTRO_OK: return "ok";
        case ENTRO_ERR_INVALID_ARG: return "invalid argument";
        case ENTRO_ERR_BUFFER_TOO_SMALL: return "buffer too small";
        case ENTRO_ERR_NONFINITE: return "tensor holds a NaN or an infinity";
        case ENTRO_ERR_CODE_TOO_LONG: return "a code length exceeds 32 bits";
        case ENTRO_ERR_CORRUPT_STREAM: return "stream, index and codebook do not agree";
        case ENTRO_ERR_CUDA: return "a CUDA call failed";
        case ENTRO_ERR_UNSUPPORTED: return "unsupported";
        case ENTRO_ERR_TOO_MANY_TENSORS: return "more tensors than the static scratch holds";
    }
    return "unknown status";
}

extern "C" uint64_t entro_index_bytes(uint64_t n, uint32_t chunk_symbols)
{
    if (chunk_symbols == 0 || chunk_symbols % kSubBlocks || chunk_symbols > ENTRO_MAX_CHUNK_SYMBOLS) return 0;
    uint64_t nc = num_chunks(n, chunk_symbols);
    return 8 * (nc + 1) + 64 * nc;
}

extern "C" uint64_t entro_encode_bound_words(uint64_t n, const entro_codebook* cb)
{
    if (!cb || cb->max_len < 1 || cb->max_len > ENTRO_MAX_CODE_LEN) return 0;
    return (n * (uint64_t)cb->max_len + 31) / 32 + ENTRO_STREAM_SLACK_WORDS;
}

extern "C" uint64_t entro_stream_words(const uint64_t* counts, const entro_codebook* cb)
{
    if (!counts || !cb || cb->nsym < 1 || cb->nsym > ENTRO_MAX_SYMBOLS) return 0;
    unsigned long long bits = 0;
    for (int k = 0; k < cb->nsym; ++k) {
        if (counts[k] && !cb->len[k]) return 0;
        bits += counts[k] * cb->len[k];
    }
    return (bits + 31) / 32 + ENTRO_STREAM_SLACK_WORDS;
}
