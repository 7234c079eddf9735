// Tensor-core linear layer for many positions at once (the first visit of a sample: the whole prompt
// goes through a partition, Section III-E / Algorithm 1 "first iteration"):
//     Y[t][r] = epilogue( sum_k W[r][k] * X[t][k] ),   W bf16 [n_rows][K],  X given as bf16 hi + lo with
//     X = hi + lo to ~16 mantissa bits, accumulation in fp32.
// The weight tile (128 rows) is the M operand of tcgen05.mma, the positions are the N operand, the
// fp32 accumulator D[128 x n_tile] lives in tensor memory.  One block = one 128-row tile x one tile of
// positions; operands arrive by TMA (128-byte swizzle, no multicast) through an mbarrier ring of 4 to 9 stages
// (as many as fit in 192 KB for the tile of positions).
// Warp 0 lane 0 issues TMA, warp 1 lane 0 issues MMAs (and warp 1 owns the TMEM allocation), warps 2..5
// read the accumulator back (tcgen05.ld, one TMEM lane = one weight row per thread) and store Y.
// Every wait is bounded in wall time; on a timeout an error word is set, the block skips the remaining
// waits, frees its tensor memory and returns.
#pragma once
#include <cuda.h>
#include <cuda_bf16.h>
#include <cuda_runtime.h>
#include <stdint.h>

namespace mdi {

constexpr int TG_BM = 128;      // weight rows per block (MMA M)
constexpr int TG_BK = 64;       // reduction elements per stage: 128 bytes, one swizzle atom
constexpr int TG_MAX_STAGES = 10;
constexpr int TG_MAX_NT = 128;  // positions per block (MMA N), a multiple of 16
constexpr int TG_THREADS = 192;
constexpr int TG_W_BYTES = TG_BM * TG_BK * 2;          // 16 KB per stage
constexpr int TG_RING_BYTES = 196608;                  // operand ring for tiles of 64 or 128 positions (4 stages at 128)
constexpr int TG_RING_BYTES_SMALL = 102400;            // for tiles of 16 (5 stages) or 32 positions (4 stages): two blocks fit on one SM,
                                                       // so GEMMs launched on different streams share SMs and overlap
constexpr int TG_RING_BYTES_PACKED = 110592;           // for 8 positions (6 stages), two blocks per SM as well
constexpr int TG_NT_PACKED = 8; // n_tile of the packed form: the hi rows and the lo rows of up to 8 positions make ONE 16-row B
                                // operand (one MMA per k-step; columns j and j + 8 of the accumulator are added in the epilogue)
constexpr size_t TG_SMEM = (size_t)TG_RING_BYTES + 1024 /* alignment slack */ + 256 /* barriers */;
__host__ __device__ inline int tg_ring_bytes(int n_tile) {
    return n_tile <= TG_NT_PACKED ? TG_RING_BYTES_PACKED : n_tile <= 32 ? TG_RING_BYTES_SMALL : TG_RING_BYTES;
}
__host__ __device__ inline size_t tg_smem_bytes(int n_tile) { return (size_t)tg_ring_bytes(n_tile) + 1024 + 256; }
// bytes of one stage: a 128 x 64 weight tile and two n_tile x 64 input tiles (hi, lo); every part 1024-byte aligned
__host__ __device__ inline int tg_stage_bytes(int n_tile) { return TG_W_BYTES + 2 * n_tile * TG_BK * 2; }
__host__ __device__ inline int tg_stages(int n_tile) {
    const int n = tg_ring_bytes(n_tile) / tg_stage_bytes(n_tile);
    return n < TG_MAX_STAGES ? n : TG_MAX_STAGES;
}
constexpr unsigned long long TG_WAIT_NS = 2000000000ull;

enum TgAct { TG_NONE = 0, TG_GELU_TANH = 1, TG_GELU_ERF = 2 };

struct TgArgs {
    int n_rows, K, T, n_tile; // weight rows, reduction length, positions, positions per block
    const float *bias;        // [n_rows] or null
    const float *resid;       // [T][ldy] or null: added to the result
    int act;                  // TgAct
    float *y;                 // [T][ldy]
    int ldy;
    int *err;                 // set to 1 when a wait gave up
    int w_tiled;              // the weights come as contiguous 128 x 64 tiles [row tile][k-block][128][64] (k_tile_weights)
    float *partial;           // split-K (gridDim.z > 1): raw partial sums [z][T][ldy]; bias/resid/act/y are then unused
    __nv_bfloat16 *out_hi, *out_lo; // optional: the result also (or, with y null, only) as two bf16 planes [T][ldy]
};

__device__ __forceinline__ uint32_t tg_smem_u32(const void *p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ unsigned long long tg_now() {
    unsigned long long t;
    asm volatile("mov.u64 %0, %%globaltimer;" : "=l"(t));
    return t;
}
__device__ __forceinline__ bool tg_try_wait(uint32_t bar, uint32_t parity) {
    uint32_t ok;
    asm volatile("{\n .reg .pred p;\n mbarrier.try_wait.parity.shared::cta.b64 p, [%1], %2;\n selp.u32 %0, 1, 0, p;\n}\n"
                 : "=r"(ok) : "r"(bar), "r"(parity) : "memory");
    return ok != 0;
}
// returns false when the wait gave up (or somebody else already did)
__device__ __noinline__ bool tg_wait(uint32_t bar, uint32_t parity, int *err) {
    unsigned long long t0 = 0;
    for (unsigned it = 0;; ++it) {
        if (tg_try_wait(bar, parity)) return true;
        if ((it & 63u) == 63u) {
            if (*(volatile int *)err) return false;
            const unsigned long long now = tg_now();
            if (t0 == 0) t0 = now;
            else if (now - t0 > TG_WAIT_NS) break;
        }
    }
    atomicExch(err, 1);
    return false;
}

// Shared-memory matrix descriptor of a K-major tile whose rows are 128 bytes, stored with the 128-byte
// swizzle (what TMA wrote): start address, stride between 8-row groups = 1024 bytes, descriptor version 1,
// layout type 2 (128-byte swizzle).  The leading-dimension offset is not used by this layout.
__device__ __forceinline__ uint64_t tg_desc(uint32_t smem_addr) {
    uint64_t d = 0;
    d |= (uint64_t)((smem_addr & 0x3FFFF) >> 4);
    d |= (uint64_t)1 << 16;
    d |= (uint64_t)(1024 >> 4) << 32;
    d |= (uint64_t)1 << 46;
    d |= (uint64_t)2 << 61;
    return d;
}
// Instruction descriptor, kind::f16: D fp32, A and B bf16, both K-major, N and M as given.
__device__ __forceinline__ uint32_t tg_idesc(int m, int n) {
    return (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(n >> 3) << 17) | ((uint32_t)(m >> 4) << 24);
}
__device__ __forceinline__ void tg_mma(uint32_t tmem_d, uint64_t adesc, uint64_t bdesc, uint32_t idesc, uint32_t accumulate) {
    asm volatile("{\n .reg .pred p;\n setp.ne.b32 p, %4, 0;\n tcgen05.mma.cta_group::1.kind::f16 [%0], %1, %2, %3, p;\n}\n"
                 ::"r"(tmem_d), "l"(adesc), "l"(bdesc), "r"(idesc), "r"(accumulate) : "memory");
}
__device__ __forceinline__ void tg_commit(uint32_t bar) {
    asm volatile("tcgen05.commit.cta_group::1.mbarrier::arrive::one.shared::cluster.b64 [%0];" ::"r"(bar) : "memory");
}
__device__ __forceinline__ void tg_tma_2d(uint32_t dst, const CUtensorMap *map, int c0, int c1, uint32_t bar) {
    asm volatile("cp.async.bulk.tensor.2d.shared::cluster.global.tile.mbarrier::complete_tx::bytes [%0], [%1, {%2, %3}], [%4];"
                 ::"r"(dst), "l"(map), "r"(c0), "r"(c1), "r"(bar) : "memory");
}

__device__ __forceinline__ float tg_apply(float v, int act) {
    if (act == TG_GELU_TANH) return 0.5f * v * (1.f + tanhf(0.7978845608028654f * (v + 0.044715f * v * v * v)));
    if (act == TG_GELU_ERF) return 0.5f * v * (1.f + erff(v * 0.7071067811865475f));
    return v;
}

// grid (ceil(n_rows / 128), ceil(T / n_tile), K splits)
__global__ void __launch_bounds__(TG_THREADS)
k_tc_gemm(const __grid_constant__ CUtensorMap tm_w, const __grid_constant__ CUtensorMap tm_xhi,
          const __grid_constant__ CUtensorMap tm_xlo, const TgArgs a) {
    extern __shared__ unsigned char tg_raw[];
    unsigned char *smem = reinterpret_cast<unsigned char *>(((uintptr_t)tg_raw + 1023) & ~(uintptr_t)1023);
    uint64_t *bars = reinterpret_cast<uint64_t *>(smem + (size_t)tg_ring_bytes(a.n_tile));
    // bars[0..S): full, bars[S..2S): empty, bars[2S]: accumulator ready; then the TMEM base address
    const int TG_STAGES = tg_stages(a.n_tile), TG_STAGE_BYTES = tg_stage_bytes(a.n_tile), TG_X_BYTES = a.n_tile * TG_BK * 2;
    uint32_t *tmem_slot = reinterpret_cast<uint32_t *>(bars + 2 * TG_MAX_STAGES + 1);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int m0 = blockIdx.x * TG_BM, t0 = blockIdx.y * a.n_tile;
    const int n_kb_all = (a.K + TG_BK - 1) / TG_BK;
    const int kb_lo = (int)((long)blockIdx.z * n_kb_all / gridDim.z), n_kb = (int)((long)(blockIdx.z + 1) * n_kb_all / gridDim.z) - kb_lo;
    const uint32_t full0 = tg_smem_u32(bars), empty0 = tg_smem_u32(bars + TG_MAX_STAGES), accbar = tg_smem_u32(bars + 2 * TG_MAX_STAGES);
    const uint32_t tmem_cols = a.n_tile <= 32 ? 32u : a.n_tile <= 64 ? 64u : 128u;

    if (tid == 0) {
        for (int s = 0; s < TG_STAGES; ++s) {
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(full0 + 8 * s) : "memory");
            asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(empty0 + 8 * s) : "memory");
        }
        asm volatile("mbarrier.init.shared::cta.b64 [%0], 1;" ::"r"(accbar) : "memory");
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 1) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(tg_smem_u32(tmem_slot)), "r"(tmem_cols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
    const uint32_t tmem_base = *tmem_slot;
    asm volatile("griddepcontrol.launch_dependents;" ::: "memory");

    if (warp == 0) {
        if (lane == 0) {
            // ---- TMA producer
            const uint32_t stage_bytes = (uint32_t)TG_STAGE_BYTES;
            bool ok = true;
            // The weights depend on nothing: the first ring of weight tiles is requested before waiting for the
            // preceding kernel (programmatic dependent launch); the inputs it produced are requested after.
            const int pre = n_kb < TG_STAGES ? n_kb : TG_STAGES;
            for (int kb = 0; kb < pre; ++kb) {
                const uint32_t full = full0 + 8 * kb, base = tg_smem_u32(smem + (size_t)kb * TG_STAGE_BYTES);
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(full), "r"(stage_bytes) : "memory");
                if (a.w_tiled) tg_tma_2d(base, &tm_w, 0, (blockIdx.x * n_kb_all + kb_lo + kb) * TG_BM, full);
                else tg_tma_2d(base, &tm_w, (kb_lo + kb) * TG_BK, m0, full);
            }
            asm volatile("griddepcontrol.wait;" ::: "memory");
            for (int kb = 0; kb < pre; ++kb) {
                const uint32_t full = full0 + 8 * kb, base = tg_smem_u32(smem + (size_t)kb * TG_STAGE_BYTES);
                tg_tma_2d(base + TG_W_BYTES, &tm_xhi, (kb_lo + kb) * TG_BK, t0, full);
                tg_tma_2d(base + TG_W_BYTES + TG_X_BYTES, &tm_xlo, (kb_lo + kb) * TG_BK, t0, full);
            }
            for (int kb = pre; kb < n_kb && ok; ++kb) {
                const int s = kb % TG_STAGES;
                if (kb >= TG_STAGES) ok = tg_wait(empty0 + 8 * s, ((kb / TG_STAGES) & 1) ^ 1, a.err);
                if (!ok) break;
                const uint32_t full = full0 + 8 * s;
                const uint32_t base = tg_smem_u32(smem + (size_t)s * TG_STAGE_BYTES);
                asm volatile("mbarrier.arrive.expect_tx.shared::cta.b64 _, [%0], %1;" ::"r"(full), "r"(stage_bytes) : "memory");
                if (a.w_tiled) tg_tma_2d(base, &tm_w, 0, (blockIdx.x * n_kb_all + kb_lo + kb) * TG_BM, full);
                else tg_tma_2d(base, &tm_w, (kb_lo + kb) * TG_BK, m0, full);
                tg_tma_2d(base + TG_W_BYTES, &tm_xhi, (kb_lo + kb) * TG_BK, t0, full);
                tg_tma_2d(base + TG_W_BYTES + TG_X_BYTES, &tm_xlo, (kb_lo + kb) * TG_BK, t0, full);
            }
        }
    } else if (warp == 1) {
        if (lane == 0) {
            // ---- MMA issuer
            const bool packed = a.n_tile == TG_NT_PACKED;
            const uint32_t idesc = tg_idesc(TG_BM, packed ? 16 : a.n_tile);
            bool ok = true;
            for (int kb = 0; kb < n_kb && ok; ++kb) {
                const int s = kb % TG_STAGES;
                ok = tg_wait(full0 + 8 * s, (kb / TG_STAGES) & 1, a.err);
                if (!ok) break;
                asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
                const uint32_t base = tg_smem_u32(smem + (size_t)s * TG_STAGE_BYTES);
#pragma unroll
                for (int k = 0; k < TG_BK / 16; ++k) {
                    const uint64_t ad = tg_desc(base + k * 32);
                    tg_mma(tmem_base, ad, tg_desc(base + TG_W_BYTES + k * 32), idesc, (kb > 0 || k > 0) ? 1u : 0u);
                    if (!packed) tg_mma(tmem_base, ad, tg_desc(base + TG_W_BYTES + TG_X_BYTES + k * 32), idesc, 1u);
                }
                tg_commit(empty0 + 8 * s);      // the stage may be refilled once these MMAs have read it
            }
            tg_commit(accbar);                  // accumulator complete (or abandoned: the epilogue then skips)
        }
    } else {
        // ---- epilogue: warps 2..5; a warp may only touch the TMEM lanes 32 * (warp % 4) .. + 31
        asm volatile("griddepcontrol.wait;" ::: "memory"); // bias / residual / partial buffers belong to earlier kernels
        const bool ok = tg_wait(accbar, 0, a.err) && *(volatile int *)a.err == 0;
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        const int lane_base = (warp & 3) * 32;
        const int row = m0 + lane_base + lane;
        const float bias = (a.bias && row < a.n_rows) ? a.bias[row] : 0.f;
        if (ok) {
            const bool packed = a.n_tile == TG_NT_PACKED;
            for (int c = 0; c < a.n_tile; c += 16) {
                uint32_t r[16];
                const uint32_t taddr = tmem_base + ((uint32_t)lane_base << 16) + (uint32_t)c;
                asm volatile("tcgen05.ld.sync.aligned.32x32b.x16.b32 {%0,%1,%2,%3,%4,%5,%6,%7,%8,%9,%10,%11,%12,%13,%14,%15}, [%16];"
                             : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]), "=r"(r[4]), "=r"(r[5]), "=r"(r[6]), "=r"(r[7]),
                               "=r"(r[8]), "=r"(r[9]), "=r"(r[10]), "=r"(r[11]), "=r"(r[12]), "=r"(r[13]), "=r"(r[14]), "=r"(r[15])
                             : "r"(taddr) : "memory");
                asm volatile("tcgen05.wait::ld.sync.aligned;" ::: "memory");
                if (packed) {
#pragma unroll
                    for (int j = 0; j < 8; ++j) r[j] = __float_as_uint(__uint_as_float(r[j]) + __uint_as_float(r[j + 8]));
                }
                if (row < a.n_rows) {
#pragma unroll
                    for (int j = 0; j < 16; ++j) {
                        const int t = (packed && j >= 8) ? a.T : t0 + c + j;
                        if (t < a.T && gridDim.z > 1) {
                            a.partial[((size_t)blockIdx.z * a.T + t) * a.ldy + row] = __uint_as_float(r[j]);
                        } else if (t < a.T) {
                            float v = __uint_as_float(r[j]) + bias;
                            if (a.resid) v += a.resid[(size_t)t * a.ldy + row];
                            v = tg_apply(v, a.act);
                            if (a.y) a.y[(size_t)t * a.ldy + row] = v;
                            if (a.out_hi) {
                                const __nv_bfloat16 h = __float2bfloat16_rn(v);
                                a.out_hi[(size_t)t * a.ldy + row] = h;
                                a.out_lo[(size_t)t * a.ldy + row] = __float2bfloat16_rn(v - __bfloat162float(h));
                            }
                        }
                    }
                }
            }
        }
    }
    asm volatile("tcgen05.fence::before_thread_sync;" ::: "memory");
    __syncthreads();
    if (warp == 1) {
        asm volatile("tcgen05.fence::after_thread_sync;" ::: "memory");
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem_base), "r"(tmem_cols) : "memory");
    }
}

// Copy of a row-major bf16 matrix [n_rows][K] as contiguous tiles [ceil(n_rows / 128)][ceil(K / 64)][128][64], zero
// outside the matrix: a block's weight tile is then one run of 16 KB in memory instead of 128 runs of 128 bytes a
// row pitch apart.  One thread per 8 elements.
__global__ void k_tile_weights(const __nv_bfloat16 *w, int n_rows, int K, __nv_bfloat16 *out, size_t n_chunks) {
    const size_t i = (size_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i >= n_chunks) return;
    const int n_kb = (K + TG_BK - 1) / TG_BK;
    const int c8 = (int)(i & 7), r = (int)((i >> 3) & (TG_BM - 1));
    const size_t tile = i >> 10;
    const int kb = (int)(tile % (size_t)n_kb), rt = (int)(tile / (size_t)n_kb);
    const int row = rt * TG_BM + r, col = kb * TG_BK + c8 * 8;
    __nv_bfloat16 v[8];
#pragma unroll
    for (int e = 0; e < 8; ++e) v[e] = (row < n_rows && col + e < K) ? w[(size_t)row * K + col + e] : __float2bfloat16_rn(0.f);
    *reinterpret_cast<uint4 *>(out + i * 8) = *reinterpret_cast<const uint4 *>(v);
}

// Host: 2-D tensor map over a row-major bf16 matrix [rows][cols] with a box of box_rows x 64 columns,
// 128-byte swizzle, zero fill outside.  cols * 2 must be a multiple of 16 bytes.  The driver's encoder is
// looked up at run time through the runtime API, so that the library does not link against the driver
// (and still loads on a machine without one).
typedef CUresult (*tg_encode_fn)(CUtensorMap *, CUtensorMapDataType, cuuint32_t, void *, const cuuint64_t *, const cuuint64_t *,
                                 const cuuint32_t *, const cuuint32_t *, CUtensorMapInterleave, CUtensorMapSwizzle,
                                 CUtensorMapL2promotion, CUtensorMapFloatOOBfill);
inline tg_encode_fn tg_encoder() {
    static tg_encode_fn fn = nullptr;
    if (!fn) {
        void *p = nullptr;
        cudaDriverEntryPointQueryResult q;
        if (cudaGetDriverEntryPoint("cuTensorMapEncodeTiled", &p, cudaEnableDefault, &q) == cudaSuccess && q == cudaDriverEntryPointSuccess)
            fn = reinterpret_cast<tg_encode_fn>(p);
    }
    return fn;
}
inline CUresult tg_make_map(CUtensorMap *map, const void *base, uint64_t rows, uint64_t cols, uint32_t box_rows) {
    const tg_encode_fn enc = tg_encoder();
    if (!enc) return CUDA_ERROR_NOT_SUPPORTED;
    cuuint64_t dims[2] = {cols, rows};
    cuuint64_t strides[1] = {cols * 2};
    cuuint32_t box[2] = {(cuuint32_t)TG_BK, box_rows};
    cuuint32_t estr[2] = {1, 1};
    return enc(map, CU_TENSOR_MAP_DATA_TYPE_BFLOAT16, 2, const_cast<void *>(base), dims, strides, box, estr,
               CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_128B,
               CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
}

} // namespace mdi
