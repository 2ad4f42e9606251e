/*
 * sifar_noalloc.cu - one all-reduce entry point that never allocates.
 *
 * The reducer of sifar_core.cu keeps its bookkeeping (the count of finished
 * CTAs that tells the last CTA it is last, call counters) in memory that
 * sifar_create() obtains from cudaMalloc.  Some callers cannot allocate at all:
 * a serving engine that handed the whole device to its own arena at start-up, or
 * a decode loop that must not meet cudaMalloc's device-wide synchronization.
 * For them the same reduction runs here with that bookkeeping in a fixed
 * file-scope device array.  The paper has no counterpart for this entry point.
 */
#include <mutex>

#include "sifar_internal.cuh"
#include "sifar_reduce.cuh"

namespace sifar {

/* Largest n the entry point accepts: 1 Mi elements per rank (2 MiB of bf16, 4 MiB of fp32). */
constexpr size_t kNoallocMaxElems = (size_t)1 << 20;
constexpr int kNoallocThreads = 256;
constexpr int kNoallocMaxDevices = 64;

/* Bookkeeping of the no-allocation reducer.  One per device that loads the library, held until exit. */
struct NoallocScratch {
    uint32_t cta_arrive;              /* CTAs of the running call that have finished; must be 0 at launch */
    uint32_t pad0[31];
    unsigned long long calls;         /* completed calls                                                  */
    unsigned long long elements;      /* elements reduced by the last completed call                      */
    uint32_t pad1[28];
};
static __device__ __align__(256) unsigned char g_noalloc_scratch[sizeof(NoallocScratch)];

struct NoallocArgs {
    const uint4 *src[kMaxRanks];
    void *out;
    unsigned long long n;
    NoallocScratch *scratch;          /* device address of g_noalloc_scratch, resolved on the host at set-up */
};

/*
 * One tile of kNoallocThreads * U 16-byte vectors per CTA, P loads in flight per
 * vector, rank-order fp32 sum, one RNE to the element type: the plain-partial
 * reducer on data that is ready in stream order (no flags, no tags).
 */
template <int DT, int P>
__global__ void __launch_bounds__(kNoallocThreads) k_reduce_noalloc(const NoallocArgs a)
{
    constexpr int U = (P <= 2) ? 4 : (P <= 4) ? 2 : 1;
    constexpr int EPV = (DT == SIFAR_BF16) ? 8 : 4;
    const size_t n = (size_t)a.n;
    const size_t nvec = n / EPV;
    const size_t base = (size_t)blockIdx.x * kNoallocThreads * U + threadIdx.x;
    uint4 x[U][P];
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t v = base + (size_t)u * kNoallocThreads;
        if (v < nvec) {
#pragma unroll
            for (int r = 0; r < P; ++r) x[u][r] = ld_slot(a.src[r] + v);
        }
    }
#pragma unroll
    for (int u = 0; u < U; ++u) {
        const size_t v = base + (size_t)u * kNoallocThreads;
        if (v < nvec) reinterpret_cast<uint4 *>(a.out)[v] = sum_vec<DT, P>(x[u], true);
    }
    /* ragged tail, fewer than EPV elements: one per thread of the last CTA */
    const size_t i = nvec * EPV + threadIdx.x;
    if (blockIdx.x == gridDim.x - 1 && i < n) {
        uint32_t w[P];
        if (DT == SIFAR_BF16) {
#pragma unroll
            for (int r = 0; r < P; ++r) w[r] = ld_relaxed_u16(reinterpret_cast<const uint16_t *>(a.src[r]) + i);
            reinterpret_cast<uint16_t *>(a.out)[i] = (uint16_t)(sum_word<DT, P>(w) & 0xFFFFu);
        } else {
#pragma unroll
            for (int r = 0; r < P; ++r) w[r] = ld_relaxed_u32(reinterpret_cast<const uint32_t *>(a.src[r]) + i);
            reinterpret_cast<uint32_t *>(a.out)[i] = sum_word<DT, P>(w);
        }
    }
    /* the last CTA out re-arms the count for the next call and books the call */
    __syncthreads();
    if (threadIdx.x == 0) {
        const uint32_t arrived = atom_add_relaxed_u32(&a.scratch->cta_arrive, 1u) + 1u;
        if (arrived == gridDim.x) {
            st_relaxed_u32(&a.scratch->cta_arrive, 0u);
            a.scratch->calls += 1ull;
            a.scratch->elements = a.n;
        }
    }
}

template <int DT>
static cudaError_t launch_noalloc_dt(int P, int grid, cudaStream_t s, const NoallocArgs &a)
{
    switch (P) {
    case 1: k_reduce_noalloc<DT, 1><<<grid, kNoallocThreads, 0, s>>>(a); break;
    case 2: k_reduce_noalloc<DT, 2><<<grid, kNoallocThreads, 0, s>>>(a); break;
    case 3: k_reduce_noalloc<DT, 3><<<grid, kNoallocThreads, 0, s>>>(a); break;
    case 4: k_reduce_noalloc<DT, 4><<<grid, kNoallocThreads, 0, s>>>(a); break;
    case 5: k_reduce_noalloc<DT, 5><<<grid, kNoallocThreads, 0, s>>>(a); break;
    case 6: k_reduce_noalloc<DT, 6><<<grid, kNoallocThreads, 0, s>>>(a); break;
    case 7: k_reduce_noalloc<DT, 7><<<grid, kNoallocThreads, 0, s>>>(a); break;
    default: k_reduce_noalloc<DT, 8><<<grid, kNoallocThreads, 0, s>>>(a); break;
    }
    return cudaGetLastError();
}

/*
 * Device address of the scratch array, per device.  In host code the name
 * g_noalloc_scratch is only a handle for the runtime, not something a kernel can
 * dereference, so the address is asked for once per device, with that device
 * current, and cached in a fixed table (no allocation here either).
 */
static std::mutex g_noalloc_mutex;
static NoallocScratch *g_noalloc_ptr[kNoallocMaxDevices];

static int noalloc_scratch(NoallocScratch **out)
{
    int dev = -1;
    SIFAR_CUDA(cudaGetDevice(&dev));
    if (dev < 0 || dev >= kNoallocMaxDevices) {
        set_error("sifar_allreduce_noalloc: device ordinal %d is outside the table of %d", dev, kNoallocMaxDevices);
        return SIFAR_ERR_INVALID;
    }
    std::lock_guard<std::mutex> lock(g_noalloc_mutex);
    if (!g_noalloc_ptr[dev]) {
        void *p = nullptr;
        SIFAR_CUDA(cudaGetSymbolAddress(&p, g_noalloc_scratch));
        g_noalloc_ptr[dev] = static_cast<NoallocScratch *>(p);
    }
    *out = g_noalloc_ptr[dev];
    return SIFAR_OK;
}

}  /* namespace sifar */

using namespace sifar;

extern "C" size_t sifar_noalloc_max_elems(void) { return kNoallocMaxElems; }

extern "C" int sifar_noalloc_counters(unsigned long long out[3])
{
    if (!out) { set_error("sifar_noalloc_counters: NULL destination"); return SIFAR_ERR_INVALID; }
    NoallocScratch *scratch = nullptr;
    int rc = noalloc_scratch(&scratch);
    if (rc) return rc;
    NoallocScratch h;
    SIFAR_CUDA(cudaDeviceSynchronize());
    SIFAR_CUDA(cudaMemcpy(&h, scratch, sizeof h, cudaMemcpyDeviceToHost));    /* to a host stack object: no allocation */
    out[0] = h.cta_arrive; out[1] = h.calls; out[2] = h.elements;
    return SIFAR_OK;
}

extern "C" int sifar_allreduce_noalloc(const void *const *rank_ptrs, int P, void *out, size_t n, int dtype,
                                       void *stream)
{
    if (P < 1 || P > kMaxRanks || (dtype != SIFAR_BF16 && dtype != SIFAR_F32) || !rank_ptrs) {
        set_error("sifar_allreduce_noalloc: need 1 <= P <= %d, dtype in {0,1} and a pointer array", kMaxRanks);
        return SIFAR_ERR_INVALID;
    }
    if (n > kNoallocMaxElems) {
        set_error("sifar_allreduce_noalloc: n = %zu exceeds the fixed limit of %zu elements per rank; "
                  "use a context (sifar_create) for larger payloads", n, kNoallocMaxElems);
        return SIFAR_ERR_INVALID;
    }
    if (n == 0) return SIFAR_OK;
    if (!out || ((uintptr_t)out & 15u)) {
        set_error("sifar_allreduce_noalloc: out must be a 16-byte aligned device pointer");
        return SIFAR_ERR_INVALID;
    }
    NoallocArgs a;
    const size_t bytes = n * elem_size(dtype);
    for (int r = 0; r < kMaxRanks; ++r) a.src[r] = nullptr;
    for (int r = 0; r < P; ++r) {
        const void *p = rank_ptrs[r];
        if (!p || ((uintptr_t)p & 15u)) {
            set_error("sifar_allreduce_noalloc: rank_ptrs[%d] must be a 16-byte aligned device pointer", r);
            return SIFAR_ERR_INVALID;
        }
        const uintptr_t x = (uintptr_t)p, y = (uintptr_t)out;
        if (x < y + bytes && y < x + bytes) {
            set_error("sifar_allreduce_noalloc: out overlaps rank_ptrs[%d]", r);
            return SIFAR_ERR_INVALID;
        }
        a.src[r] = static_cast<const uint4 *>(p);
    }
    a.out = out;
    a.n = n;
    int rc = noalloc_scratch(&a.scratch);
    if (rc) return rc;
    cudaStream_t s = (cudaStream_t)stream;
    /* the count of finished CTAs must start at zero even if an earlier call never completed */
    SIFAR_CUDA(cudaMemsetAsync(&a.scratch->cta_arrive, 0, sizeof(uint32_t), s));
    const int per_thread = P <= 2 ? 4 : P <= 4 ? 2 : 1;
    const size_t per_cta = (size_t)kNoallocThreads * per_thread;
    size_t grid = (bytes / 16 + per_cta - 1) / per_cta;
    if (grid < 1) grid = 1;
    cudaError_t err = (dtype == SIFAR_BF16) ? launch_noalloc_dt<SIFAR_BF16>(P, (int)grid, s, a)
                                            : launch_noalloc_dt<SIFAR_F32>(P, (int)grid, s, a);
    SIFAR_CUDA(err);
    return SIFAR_OK;
}
