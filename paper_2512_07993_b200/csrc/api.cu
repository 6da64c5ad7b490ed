// Workspace management, argument checks and error reporting of the SkipKV C ABI.
#include <cstdio>
#include <cstring>

#include "common.cuh"
#include "tc.cuh"

namespace skipkv {

static thread_local char g_err[256] = "";

void set_error_text(const char* msg) { std::snprintf(g_err, sizeof(g_err), "%s", msg); }

int cuda_fail(cudaError_t e) {
    std::snprintf(g_err, sizeof(g_err), "%s: %s", cudaGetErrorName(e), cudaGetErrorString(e));
    return SKIPKV_ERR_CUDA;
}

int num_sms() {
    static thread_local int cached_dev = -1, cached = 0;
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess) return 148;
    if (dev != cached_dev) {
        int n = 0;
        if (cudaDeviceGetAttribute(&n, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || n <= 0) n = 148;
        cached = n;
        cached_dev = dev;
    }
    return cached;
}

// cuTensorMapEncodeTiled is looked up through the runtime so the library does not link libcuda.
typedef CUresult (*EncodeTiledFn)(CUtensorMap*, CUtensorMapDataType, cuuint32_t, void*, const cuuint64_t*,
                                  const cuuint64_t*, const cuuint32_t*, const cuuint32_t*, CUtensorMapInterleave,
                                  CUtensorMapSwizzle, CUtensorMapL2promotion, CUtensorMapFloatOOBfill);

static EncodeTiledFn encode_tiled_fn() {
    static EncodeTiledFn fn = [] {
        void* p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) != cudaSuccess ||
            q != cudaDriverEntryPointSuccess)
            p = nullptr;
        return reinterpret_cast<EncodeTiledFn>(p);
    }();
    return fn;
}

static int encode(CUtensorMap* out, const void* base, int rank, const cuuint64_t* dims, const cuuint64_t* strides,
                  const cuuint32_t* box) {
    EncodeTiledFn fn = encode_tiled_fn();
    if (!fn) {
        set_error_text("cuTensorMapEncodeTiled is not available from this driver");
        return SKIPKV_ERR_CUDA;
    }
    const cuuint32_t estr[3] = {1, 1, 1};
    const CUresult r = fn(out, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, cuuint32_t(rank), const_cast<void*>(base), dims,
                          strides, box, estr, CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B,
                          CU_TENSOR_MAP_L2_PROMOTION_L2_128B, CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) {
        char msg[96];
        std::snprintf(msg, sizeof(msg), "cuTensorMapEncodeTiled failed with CUresult %d", int(r));
        set_error_text(msg);
        return SKIPKV_ERR_CUDA;
    }
    return SKIPKV_OK;
}

int tmap_rows(CUtensorMap* out, const void* base, uint64_t rows, uint32_t box_rows) {
    const cuuint64_t dims[2] = {cuuint64_t(kHeadDim), rows};
    const cuuint64_t strides[1] = {cuuint64_t(kRowBytes)};
    const cuuint32_t box[2] = {64, box_rows};
    return encode(out, base, 2, dims, strides, box);
}

int tmap_qwin(CUtensorMap* out, const void* base, uint64_t heads, uint32_t window, uint32_t box_w, uint32_t box_heads) {
    const cuuint64_t dims[3] = {cuuint64_t(kHeadDim), window, heads};
    const cuuint64_t strides[2] = {cuuint64_t(kRowBytes), cuuint64_t(kRowBytes) * window};
    const cuuint32_t box[3] = {64, box_w, box_heads};
    return encode(out, base, 3, dims, strides, box);
}

int check_shape(const skipkv_shape* s) {
    if (!s) return SKIPKV_ERR_INVALID_ARG;
    if (s->batch <= 0 || s->n_q_heads <= 0 || s->n_kv_heads <= 0 || s->window <= 0 || s->max_sent < 0 ||
        s->max_cap <= 0 || s->d_model < 0 || s->total_rows <= 0)
        return SKIPKV_ERR_INVALID_ARG;
    if (!s->slab_off || !s->cap) return SKIPKV_ERR_INVALID_ARG;
    if (s->head_dim != kHeadDim) return SKIPKV_ERR_UNSUPPORTED;
    if (s->n_q_heads % s->n_kv_heads != 0) return SKIPKV_ERR_UNSUPPORTED;
    const int group = s->n_q_heads / s->n_kv_heads;
    if (group > kMaxGroup || group * s->window > kMaxQRows) return SKIPKV_ERR_UNSUPPORTED;
    if ((s->window + 128 / group - 1) / (128 / group) > kMaxQueryBlocks) return SKIPKV_ERR_UNSUPPORTED;
    if (s->total_rows > int64_t(0x7fffffff) - 256) return SKIPKV_ERR_UNSUPPORTED;
    if (s->d_model % 8 != 0) return SKIPKV_ERR_UNSUPPORTED;
    if (int64_t(s->batch) * s->n_kv_heads > (1 << 20)) return SKIPKV_ERR_UNSUPPORTED;
    return SKIPKV_OK;
}

__global__ void ws_set_word_kernel(uint32_t* p, uint32_t v) { *p = v; }

// One warp waits, with the workspace's wait limit, for a barrier phase that nothing will ever complete.
__global__ void __launch_bounds__(32) wait_probe_kernel(Header* hdr) {
    __shared__ __align__(8) uint64_t bar;
    if (threadIdx.x == 0) { mbar_init(&bar, 1); mbar_fence_init(); }
    __syncwarp();
    const uint32_t limit = load_wait_limit(hdr);
    const bool ok = mbar_wait(&bar, 0u, limit);
    if (!ok && threadIdx.x == 0) atomicOr(&hdr->status, SKIPKV_STATUS_COPY_TIMEOUT);
}

__global__ void ws_clear_kernel(uint32_t* p, size_t n_words) {
    for (size_t i = blockIdx.x * size_t(blockDim.x) + threadIdx.x; i < n_words; i += size_t(gridDim.x) * blockDim.x)
        p[i] = 0u;
}

}  // namespace skipkv

using namespace skipkv;

extern "C" {

int skipkv_workspace_bytes(const skipkv_shape* shape, size_t* bytes) {
    if (!bytes) return SKIPKV_ERR_INVALID_ARG;
    // slab_off / cap are not needed to size the workspace
    if (!shape) return SKIPKV_ERR_INVALID_ARG;
    skipkv_shape s = *shape;
    static const int64_t dummy_off = 0;
    static const int32_t dummy_cap = 0;
    if (!s.slab_off) s.slab_off = &dummy_off;
    if (!s.cap) s.cap = &dummy_cap;
    if (int rc = check_shape(&s)) return rc;
    *bytes = make_layout(s).total;
    return SKIPKV_OK;
}

int skipkv_workspace_init(const skipkv_shape* shape, void* ws, void* stream) {
    if (int rc = check_shape(shape)) return rc;
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255)) return SKIPKV_ERR_WORKSPACE;
    const WsLayout L = make_layout(*shape);
    // header + every counter region (everything before the decode partials)
    const size_t words = L.dec_part / 4;
    ws_clear_kernel<<<592, 256, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<uint32_t*>(ws), words);
    SKIPKV_CUDA(cudaGetLastError());
    return SKIPKV_OK;
}

int skipkv_set_wait_limit(void* ws, uint32_t polls, void* stream) {
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255)) return SKIPKV_ERR_WORKSPACE;
    ws_set_word_kernel<<<1, 1, 0, static_cast<cudaStream_t>(stream)>>>(&static_cast<Header*>(ws)->wait_limit, polls);
    SKIPKV_CUDA(cudaGetLastError());
    return SKIPKV_OK;
}

int skipkv_wait_probe(void* ws, void* stream) {
    if (!ws || (reinterpret_cast<uintptr_t>(ws) & 255)) return SKIPKV_ERR_WORKSPACE;
    wait_probe_kernel<<<1, 32, 0, static_cast<cudaStream_t>(stream)>>>(static_cast<Header*>(ws));
    SKIPKV_CUDA(cudaGetLastError());
    return SKIPKV_OK;
}

int skipkv_status(void* ws, void* stream, uint32_t* status_bits) {
    if (!ws) return SKIPKV_ERR_WORKSPACE;
    uint32_t bits = 0;
    cudaStream_t st = static_cast<cudaStream_t>(stream);
    SKIPKV_CUDA(cudaMemcpyAsync(&bits, ws, sizeof(bits), cudaMemcpyDeviceToHost, st));
    SKIPKV_CUDA(cudaStreamSynchronize(st));
    if (bits) {
        SKIPKV_CUDA(cudaMemsetAsync(ws, 0, sizeof(bits), st));
        SKIPKV_CUDA(cudaStreamSynchronize(st));
    }
    if (status_bits) *status_bits = bits;
    if (bits & (SKIPKV_STATUS_COMPACT_TIMEOUT | SKIPKV_STATUS_COPY_TIMEOUT)) return SKIPKV_ERR_TIMEOUT;
    if (bits & SKIPKV_STATUS_BAD_TABLE) return SKIPKV_ERR_INVALID_ARG;
    return SKIPKV_OK;
}

const char* skipkv_last_cuda_error(void) { return g_err; }

}  // extern "C"
