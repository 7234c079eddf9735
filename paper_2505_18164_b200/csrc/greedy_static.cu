// Greedy token choice that allocates nothing: a variant of the output layer's two-level argmax whose
// per-block partial results live in a fixed device array instead of memory obtained from cudaMalloc.
//
// Who needs this.  Some callers of the library are not allowed to allocate device memory at the point
// where they pick tokens: a serving loop that has handed all of the device's memory to its own pool and
// must not disturb it, a latency-critical section where an implicit device synchronisation (cudaMalloc
// and cudaFree may cause one) is unacceptable, or a process whose allocator is owned by another
// component.  They hold the logits themselves and only need the winning index per row.
#include "mdi.h"

#include <cuda_runtime.h>

#include <cstdio>

void mdi_internal_set_error(const char *text); // mdi.cu: text returned by mdi_last_error(NULL)

namespace {

constexpr int GS_MAX_ROWS = 64;        // rows (samples) per call
constexpr int GS_COLS_PER_BLOCK = 1024;
constexpr int GS_MAX_BLOCKS = 256;     // per row: at most 262144 columns
constexpr int GS_THREADS = 256;

struct GsPartial { float v; int i; };
struct GsScratch {
    GsPartial part[GS_MAX_ROWS][GS_MAX_BLOCKS]; // best (value, index) of each block of columns
    unsigned ticket[GS_MAX_ROWS];               // blocks of the row that have finished; must be zero at launch
};

// Shared by every call on this device and held until the process exits (about 128 KB per GPU that loads
// the library).  In host code this name is only a stand-in; the device address comes from
// cudaGetSymbolAddress (see gs_scratch_for_current_device).
static __device__ __align__(256) GsScratch g_gs_scratch;

__device__ __forceinline__ bool gs_better(float v, int i, float bv, int bi) { return v > bv || (v == bv && i < bi); }

// grid (blocks per row, rows).  Each block scans GS_COLS_PER_BLOCK columns of one row; the block that
// finishes last for a row merges that row's partials.  Ties go to the lowest index.
__global__ void __launch_bounds__(GS_THREADS) k_greedy_static(const float *logits, int n_cols, int *out, GsScratch *sc) {
    __shared__ float sv[GS_THREADS / 32];
    __shared__ int si[GS_THREADS / 32];
    __shared__ bool is_last;
    const int row = blockIdx.y, blk = blockIdx.x, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float *x = logits + (size_t)row * n_cols;
    float bv = -INFINITY;
    int bi = 0x7fffffff;
    const int c0 = blk * GS_COLS_PER_BLOCK, c1 = min(n_cols, c0 + GS_COLS_PER_BLOCK);
    for (int c = c0 + tid; c < c1; c += GS_THREADS) {
        const float v = x[c];
        if (gs_better(v, c, bv, bi)) { bv = v; bi = c; }
    }
    auto warp_best = [&]() {
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const float v = __shfl_xor_sync(0xffffffffu, bv, o);
            const int i = __shfl_xor_sync(0xffffffffu, bi, o);
            if (gs_better(v, i, bv, bi)) { bv = v; bi = i; }
        }
    };
    auto block_best = [&]() { // result valid in thread 0
        warp_best();
        if (lane == 0) { sv[warp] = bv; si[warp] = bi; }
        __syncthreads();
        if (warp == 0) {
            bv = lane < GS_THREADS / 32 ? sv[lane] : -INFINITY;
            bi = lane < GS_THREADS / 32 ? si[lane] : 0x7fffffff;
            warp_best();
        }
        __syncthreads();
    };
    block_best();
    if (tid == 0) {
        sc->part[row][blk].v = bv;
        sc->part[row][blk].i = bi;
        __threadfence();
        is_last = atomicAdd(&sc->ticket[row], 1u) == gridDim.x - 1;
    }
    __syncthreads();
    if (!is_last) return;
    __threadfence();
    bv = -INFINITY;
    bi = 0x7fffffff;
    for (int b = tid; b < (int)gridDim.x; b += GS_THREADS) {
        const float v = __ldcg(&sc->part[row][b].v);
        const int i = __ldcg(&sc->part[row][b].i);
        if (gs_better(v, i, bv, bi)) { bv = v; bi = i; }
    }
    block_best();
    if (tid == 0) {
        out[row] = bi;
        sc->ticket[row] = 0u;
    }
}

// Device address of the scratch array on the current device, looked up once per device.
GsScratch *g_gs_ptr[64] = {nullptr};

int gs_fail(int code, const char *text) {
    mdi_internal_set_error(text);
    return code;
}

int gs_scratch_for_current_device(GsScratch **out) {
    int dev = 0;
    if (cudaGetDevice(&dev) != cudaSuccess || dev < 0 || dev >= 64) return gs_fail(MDI_ERR_CUDA, "mdi_greedy_argmax_static: no usable current CUDA device");
    if (!g_gs_ptr[dev]) {
        GsScratch *p = nullptr;
        const cudaError_t e = cudaGetSymbolAddress((void **)&p, g_gs_scratch);
        if (e != cudaSuccess || !p) {
            char buf[256];
            snprintf(buf, sizeof buf, "mdi_greedy_argmax_static: cudaGetSymbolAddress failed: %s", cudaGetErrorString(e));
            return gs_fail(MDI_ERR_CUDA, buf);
        }
        g_gs_ptr[dev] = p;
    }
    *out = g_gs_ptr[dev];
    return MDI_OK;
}

} // namespace

extern "C" int mdi_greedy_argmax_static(const float *logits_dev, int n_rows, int n_cols, int32_t *out_dev, void *stream) {
    if (!logits_dev || !out_dev) return gs_fail(MDI_ERR_ARG, "mdi_greedy_argmax_static: null pointer");
    if (n_rows < 1 || n_cols < 1) return gs_fail(MDI_ERR_ARG, "mdi_greedy_argmax_static: n_rows and n_cols must be positive");
    if (n_rows > GS_MAX_ROWS || n_cols > GS_MAX_BLOCKS * GS_COLS_PER_BLOCK) {
        char buf[256];
        snprintf(buf, sizeof buf, "mdi_greedy_argmax_static: %d x %d exceeds the fixed scratch (at most %d rows of %d columns)", n_rows,
                 n_cols, GS_MAX_ROWS, GS_MAX_BLOCKS * GS_COLS_PER_BLOCK);
        return gs_fail(MDI_ERR_SHAPE, buf);
    }
    GsScratch *sc = nullptr;
    int rc = gs_scratch_for_current_device(&sc);
    if (rc != MDI_OK) return rc;
    cudaStream_t st = (cudaStream_t)stream;
    // the array keeps whatever the previous call left: the counters must start at zero
    cudaError_t e = cudaMemsetAsync(sc->ticket, 0, sizeof(unsigned) * GS_MAX_ROWS, st);
    if (e == cudaSuccess) {
        const dim3 grid((n_cols + GS_COLS_PER_BLOCK - 1) / GS_COLS_PER_BLOCK, n_rows);
        k_greedy_static<<<grid, GS_THREADS, 0, st>>>(logits_dev, n_cols, out_dev, sc);
        e = cudaGetLastError();
    }
    if (e != cudaSuccess) {
        char buf[256];
        snprintf(buf, sizeof buf, "mdi_greedy_argmax_static: %s", cudaGetErrorString(e));
        return gs_fail(MDI_ERR_CUDA, buf);
    }
    return MDI_OK;
}
