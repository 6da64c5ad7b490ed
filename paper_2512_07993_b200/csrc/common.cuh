// Shared host/device helpers of the SkipKV CUDA library (sm_100a only).
#pragma once

#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stddef.h>
#include <stdint.h>

#include "skipkv.h"

namespace skipkv {

constexpr int kHeadDim = 128;
constexpr int kRowBytes = kHeadDim * 2;       // one bf16 K or V row
constexpr int kMaxGroup = 8;                  // query heads per KV head
constexpr int kMaxQRows = 512;                // group * window

// ---------------------------------------------------------------------------------------
// Workspace layout.  All offsets are multiples of 256 bytes from the workspace base.
// ---------------------------------------------------------------------------------------
struct Header {                // first 256 bytes of the workspace
    uint32_t status;           // SKIPKV_STATUS_* bits
    uint32_t compact_ticket;   // dynamic segment scheduler of the compaction kernel
    uint32_t wait_limit;       // polls a bounded device wait makes before it gives up; 0 = kDefaultWaitLimit
    uint32_t pad[61];
};
constexpr uint32_t kDefaultWaitLimit = 1u << 22;

struct WsLayout {
    size_t header;
    size_t cp_nseg;        // int32  [slabs]              segments per stream
    size_t cp_loaded;      // uint32 [2*slabs]            segments whose loads are complete
    size_t cp_nruns;       // int32  [slabs]
    size_t cp_run_src;     // int32  [slabs][max_sent]    first source token of a run
    size_t cp_run_dst;     // int32  [slabs][max_sent+1]  first destination token; [nruns] = new_len
    size_t dec_cnt;        // uint32 [slabs]              partials that arrived (self-resetting)
    size_t dec_part;       // float  [max_ctas + slabs][group][130]
    size_t sc_part;        // float2 [(max_ctas + slabs) * 4][sc_rb * 128]  (max, sum) of a CTA's part of a slab
    size_t sc_tokimp;      // float  [slabs][max_cap]
    size_t sc_vsum;        // float  [slabs][max_sent][128]  per-sentence sums of key rows
    size_t sc_vbar_hi;     // bf16   [slabs][max_sent][128]  normalised mean key, high part
    size_t sc_vbar_lo;     // bf16   [slabs][max_sent][128]  and the rounding remainder
    size_t sc_z;           // float  [slabs][max_sent]
    size_t cp_part;        // int32  [slabs][1 + 3*kMaxPartial]  partly kept sentences: count, then (begin, end, dst)
    size_t tr_inv;         // float  [slabs][max_cap]  token redundancy: 1 / (|K_t| + eps)
    size_t tr_z;           // float  [slabs][max_cap]  token redundancy: row sums of exp(G)
    size_t total;
    int slabs, group, qrows, dec_max_ctas;
    int sc_wb;             // window positions per query block: floor(128 / group)
    int sc_rb;             // query blocks per group: ceil(window / sc_wb)
};

constexpr int kDecMaxCtas = 1024;     // upper bound of the persistent grids
constexpr int kMaxQueryBlocks = 4;
constexpr int kMaxPartial = 4;        // partly kept sentences per slab that one compaction call can carry

inline size_t align256(size_t x) { return (x + 255) & ~size_t(255); }

inline WsLayout make_layout(const skipkv_shape& s) {
    WsLayout L{};
    L.slabs = s.batch * s.n_kv_heads;
    L.group = s.n_q_heads / s.n_kv_heads;
    L.qrows = L.group * s.window;
    L.sc_wb = 128 / (L.group > 0 ? L.group : 1);
    L.sc_rb = (s.window + L.sc_wb - 1) / L.sc_wb;
    L.dec_max_ctas = kDecMaxCtas;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t r = o; o = align256(o + bytes); return r; };
    const size_t slabs = L.slabs, ms = s.max_sent > 0 ? s.max_sent : 1;
    L.header = take(sizeof(Header));
    L.cp_nseg = take(slabs * 4);
    L.cp_loaded = take(slabs * 2 * 4);
    L.cp_nruns = take(slabs * 4);
    L.cp_run_src = take(slabs * ms * 4);
    L.cp_run_dst = take(slabs * (ms + 1) * 4);
    L.dec_cnt = take(slabs * 4);
    L.dec_part = take((size_t(L.dec_max_ctas) + slabs) * L.group * 130 * 4);
    L.sc_part = take((size_t(L.dec_max_ctas) + slabs) * 4 * size_t(L.sc_rb) * 128 * 8);
    L.sc_tokimp = take(slabs * size_t(s.max_cap > 0 ? s.max_cap : 1) * 4);
    L.sc_vsum = take(slabs * ms * kHeadDim * 4);
    L.sc_vbar_hi = take(slabs * ms * kHeadDim * 2);
    L.sc_vbar_lo = take(slabs * ms * kHeadDim * 2);
    L.sc_z = take(slabs * ms * 4);
    L.cp_part = take(slabs * (1 + 3 * kMaxPartial) * 4);
    L.tr_inv = take(slabs * size_t(s.max_cap > 0 ? s.max_cap : 1) * 4);
    L.tr_z = take(slabs * size_t(s.max_cap > 0 ? s.max_cap : 1) * 4);
    L.total = o;
    return L;
}

int check_shape(const skipkv_shape* s);          // SKIPKV_OK or an error code
int cuda_fail(cudaError_t e);                    // records the message, returns SKIPKV_ERR_CUDA
void set_error_text(const char* msg);            // text returned by skipkv_last_cuda_error
int num_sms();

#define SKIPKV_CUDA(expr)                                            \
    do {                                                             \
        cudaError_t e__ = (expr);                                    \
        if (e__ != cudaSuccess) return ::skipkv::cuda_fail(e__);     \
    } while (0)

// ---------------------------------------------------------------------------------------
// Device helpers
// ---------------------------------------------------------------------------------------
#ifdef __CUDACC__

// Programmatic dependent launch between the kernels of one call: a kernel lets its successor's CTAs start early
// (pdl_trigger, a no-op without a dependent), and the successor waits (pdl_wait, a no-op when launched normally)
// until the predecessor grid has completed and its writes are visible, before it touches anything that grid wrote.
__device__ __forceinline__ void pdl_trigger() { asm volatile("griddepcontrol.launch_dependents;" ::: "memory"); }
__device__ __forceinline__ void pdl_wait() { asm volatile("griddepcontrol.wait;" ::: "memory"); }

// host: launch `kernel` on `st` as a programmatic dependent of the kernel enqueued before it
template <typename... KArgs, typename... Args>
inline cudaError_t launch_dependent(void (*kernel)(KArgs...), dim3 grid, dim3 block, size_t smem, cudaStream_t st,
                                    Args... args) {
    cudaLaunchConfig_t cfg{};
    cfg.gridDim = grid;
    cfg.blockDim = block;
    cfg.dynamicSmemBytes = smem;
    cfg.stream = st;
    cudaLaunchAttribute attr{};
    attr.id = cudaLaunchAttributeProgrammaticStreamSerialization;
    attr.val.programmaticStreamSerializationAllowed = 1;
    cfg.attrs = &attr;
    cfg.numAttrs = 1;
    return cudaLaunchKernelEx(&cfg, kernel, KArgs(args)...);
}

__device__ __forceinline__ size_t slab_row0(const int64_t* slab_off, const int32_t* cap, int Hk, int b, int h) {
    return size_t(slab_off[b]) * Hk + size_t(h) * cap[b];
}

__device__ __forceinline__ float bf16lo(uint32_t x) { return __uint_as_float(x << 16); }
__device__ __forceinline__ float bf16hi(uint32_t x) { return __uint_as_float(x & 0xffff0000u); }
__device__ __forceinline__ float2 bf16x2_to_f2(uint32_t x) { return make_float2(bf16lo(x), bf16hi(x)); }

__device__ __forceinline__ uint32_t smem_u32(const void* p) {
    return static_cast<uint32_t>(__cvta_generic_to_shared(p));
}

// ---- mbarrier + bulk asynchronous copies (TMA engine, untiled form) -------------------
__device__ __forceinline__ void mbar_init(uint64_t* bar, uint32_t count) {
    asm volatile("mbarrier.init.shared::cta.b64 [%0], %1;" ::"r"(smem_u32(bar)), "r"(count) : "memory");
}
__device__ __forceinline__ void mbar_fence_init() {
    asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
}
__device__ __forceinline__ void mbar_expect_tx(uint64_t* bar, uint32_t bytes) {
    asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(smem_u32(bar)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void mbar_arrive(uint64_t* bar) {
    asm volatile("mbarrier.arrive.shared::cta.b64 _, [%0];" ::"r"(smem_u32(bar)) : "memory");
}
__device__ __forceinline__ bool mbar_try_wait(uint64_t* bar, uint32_t parity) {
    uint32_t ok;
    asm volatile(
        "{\n\t.reg .pred p;\n\t"
        "mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n\t"
        "selp.u32 %0, 1, 0, p;\n\t}"
        : "=r"(ok)
        : "r"(smem_u32(bar)), "r"(parity)
        : "memory");
    return ok != 0;
}
// Bounded wait: returns false if the phase did not complete within the limit.  The first probe is
// inline (the common case: the data is already there); the retry loop is kept out of line.
static __device__ __noinline__ bool mbar_wait_slow(uint64_t* bar, uint32_t parity, uint32_t limit) {
    for (uint32_t i = 0; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i > 64) __nanosleep(64);
    }
    return false;
}
__device__ __forceinline__ bool mbar_wait(uint64_t* bar, uint32_t parity, uint32_t limit = (1u << 22)) {
    if (mbar_try_wait(bar, parity)) return true;
    return mbar_wait_slow(bar, parity, limit);
}
// global -> shared, completion counted in bytes on an mbarrier.  16-byte aligned, size % 16 == 0.
__device__ __forceinline__ void bulk_g2s(void* smem_dst, const void* gsrc, uint32_t bytes, uint64_t* bar) {
    asm volatile(
        "cp.async.bulk.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1], %2, [%3];" ::"r"(
            smem_u32(smem_dst)),
        "l"(gsrc), "r"(bytes), "r"(smem_u32(bar))
        : "memory");
}
// shared -> global, tracked by the issuing thread's bulk async-group.
__device__ __forceinline__ void bulk_s2g(void* gdst, const void* smem_src, uint32_t bytes) {
    asm volatile("cp.async.bulk.global.shared::cta.bulk_group [%0], [%1], %2;" ::"l"(gdst),
                 "r"(smem_u32(smem_src)), "r"(bytes)
                 : "memory");
}
__device__ __forceinline__ void bulk_commit() { asm volatile("cp.async.bulk.commit_group;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_all() { asm volatile("cp.async.bulk.wait_group 0;" ::: "memory"); }
__device__ __forceinline__ void bulk_wait_read_all() {
    asm volatile("cp.async.bulk.wait_group.read 0;" ::: "memory");
}
__device__ __forceinline__ void fence_proxy_async() { asm volatile("fence.proxy.async;" ::: "memory"); }
// The same for shared memory only (generic writes to shared memory that the tensor core or a bulk copy reads next).
__device__ __forceinline__ void fence_proxy_async_smem() { asm volatile("fence.proxy.async.shared::cta;" ::: "memory"); }

// The wait limit a workspace carries (skipkv_set_wait_limit); 0 stands for the default.
__device__ __forceinline__ uint32_t load_wait_limit(const Header* hdr) {
    const uint32_t v = *reinterpret_cast<const volatile uint32_t*>(&hdr->wait_limit);
    return v ? v : kDefaultWaitLimit;
}

// Bounded wait of one role of a warp-specialised CTA: gives up after `limit` polls, or as soon as another role
// of the CTA has flagged a failure; on expiry it flags the failure itself (status word + the CTA's abort flag).
// The first probe is inline (the common case: the phase is already complete); the retry loop is kept out of line.
static __device__ __noinline__ bool role_wait_slow(uint64_t* bar, uint32_t parity, uint32_t limit, int* abort_flag, uint32_t* status) {
    if (*reinterpret_cast<volatile int*>(abort_flag)) return false;
    for (uint32_t i = 0; i < limit; ++i) {
        if (mbar_try_wait(bar, parity)) return true;
        if (i > 64) {
            __nanosleep(64);
            if ((i & 255) == 0 && *reinterpret_cast<volatile int*>(abort_flag)) return false;
        }
    }
    atomicOr(status, SKIPKV_STATUS_COPY_TIMEOUT);
    *reinterpret_cast<volatile int*>(abort_flag) = 1;
    return false;
}
__device__ __forceinline__ bool role_wait(uint64_t* bar, uint32_t parity, uint32_t limit, int* abort_flag, uint32_t* status) {
    if (mbar_try_wait(bar, parity)) return true;
    return role_wait_slow(bar, parity, limit, abort_flag, status);
}

// Exclusive prefix of count(0..n-1) into pref[0..n] (pref[n] = total) by a whole CTA of kThreads threads; every thread
// owns a contiguous block of indices.  wsum: kThreads / 32 words of shared memory.  Holds two CTA barriers; the
// first one also publishes whatever the caller set up in shared memory before the call.
template <int kThreads, typename F>
__device__ __forceinline__ void cta_prefix(int n, F count, int* pref, uint32_t* wsum) {
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int per = (n + kThreads - 1) / kThreads;
    const int s0 = min(tid * per, n), s1 = min(s0 + per, n);
    uint32_t local = 0;
    for (int s = s0; s < s1; ++s) local += uint32_t(count(s));
    uint32_t inc = local;
#pragma unroll
    for (int d = 1; d < 32; d <<= 1) {
        const uint32_t x = __shfl_up_sync(0xffffffffu, inc, d);
        if (lane >= d) inc += x;
    }
    if (lane == 31) wsum[warp] = inc;
    __syncthreads();
    uint32_t base = 0;
    for (int w = 0; w < warp; ++w) base += wsum[w];
    uint32_t run = base + inc - local;
    for (int s = s0; s < s1; ++s) {
        pref[s] = int(run);
        run += uint32_t(count(s));
    }
    if (tid == kThreads - 1) pref[n] = int(run);
    __syncthreads();
}

#endif  // __CUDACC__

}  // namespace skipkv
