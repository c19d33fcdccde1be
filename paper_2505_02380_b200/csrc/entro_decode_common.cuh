// Shared-memory window, constants and small load helpers of the decode kernels.
// Included by entro_decode.cu only.
#pragma once

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

// Checked build (-DENTRO_CHECKED): every access whose address the kernel works out by hand
// (shared-window addresses of table cells, ring words, index slots and x; the places of the
// bulk copies; the output) is tested first; a violation is counted in g_check_violations
// and the access is left out (reads give 0).  Nothing traps.  In the ordinary build
// ENTRO_CHECK(ok) is the constant false and the tests vanish.
#ifdef ENTRO_CHECKED
__device__ unsigned int g_check_violations;
__device__ __forceinline__ bool check_failed(bool ok)
{
    if (!ok) atomicAdd(&g_check_violations, 1u);
    return !ok;
}
#define ENTRO_CHECK(ok) check_failed(ok)
#else
#define ENTRO_CHECK(ok) false
#endif

// Does [addr, addr + bytes) lie inside this CTA's dynamic shared memory, aligned to `bytes`?
__device__ __forceinline__ bool smem_ok(uint32_t addr, uint32_t bytes)
{
    uint32_t size;
    asm("mov.u32 %0, %%dynamic_smem_size;" : "=r"(size));
    return (addr & (bytes - 1u)) == 0u && addr >= kSmemBase && addr + bytes <= kSmemBase + size;
}

// 32-bit word at a shared-window address.
__device__ __forceinline__ uint32_t lds32(uint32_t addr)
{
    if (ENTRO_CHECK(smem_ok(addr, 4u))) return 0u;
    uint32_t v;
    asm volatile("ld.shared.b32 %0, [%1];" : "=r"(v) : "r"(addr));
    return v;
}

// Shared-memory bytes of the lookup tables for a K-bit eight-symbol table.
__host__ __device__ constexpr uint32_t lut_bytes(int K)
{
    return (17u << K) + 4u * kExpEntriesMin > 65536u ? (17u << K) + 4u * kExpEntriesMin : 65536u;
}

}  // namespace
}  // namespace entro
