// Helper kernels of the tensor-core first visit (whole prompt through a partition): everything around
// the GEMMs of tc_gemm.cuh.  Activations are fp32 [position][feature]; the GEMM inputs are written as two
// bf16 planes (hi, lo) with x = hi + lo to about 16 mantissa bits, so that the tensor cores lose nothing
// that matters against the fp32 CUDA-core path.
#pragma once
#include "step_kernels.cuh"

namespace mdi {

constexpr int PF_THREADS = 512;

__device__ __forceinline__ void pf_split_store(__nv_bfloat16 *hi, __nv_bfloat16 *lo, size_t i, float v) {
    const __nv_bfloat16 h = __float2bfloat16_rn(v);
    hi[i] = h;
    lo[i] = __float2bfloat16_rn(v - __bfloat162float(h));
}

// x[t][:] = wte[tok[t]][:] (+ wpe[pos0 + t][:]);  grid (T)
template <typename WT>
__global__ void k_pf_embed(const WT *wte, const WT *wpe, int d, int vocab, const int *tok, const int *pos, int slot, float *x) {
    pdl_launch_dependents();
    pdl_wait();
    const int t = blockIdx.x;
    const int id = min(max(tok[t], 0), vocab - 1);
    const int p = pos[slot] + t;
    for (int e = threadIdx.x; e < d; e += blockDim.x) {
        float v = __bfloat162float(wte[(size_t)id * d + e]);
        if (wpe) v += __bfloat162float(wpe[(size_t)p * d + e]);
        x[(size_t)t * d + e] = v;
    }
}

// Row t of the input is x[t][:] (+ bias + the split-K partial sums of the GEMM that produced it, added in a
// fixed order; the completed row is then stored to x_store, which becomes the residual stream).  Followed by
// LayerNorm / RMSNorm (skipped when gamma is null) and the hi/lo split (skipped when hi is null).
// grid (T, column slices): more than one slice only for the purely element-wise uses (no norm).  A thread keeps up
// to PF_VPT float4 of its row in registers from the first load to the last store (rows of up to 16384 elements);
// longer rows go through the plain loops at the end.
constexpr int PF_VPT = 4;
__device__ __forceinline__ void pf_split_store4(__nv_bfloat16 *hi, __nv_bfloat16 *lo, size_t i, const float4 v) {
    const float f[4] = {v.x, v.y, v.z, v.w};
    uint16_t h[4], l[4];
#pragma unroll
    for (int e = 0; e < 4; ++e) {
        const __nv_bfloat16 hb = __float2bfloat16_rn(f[e]);
        h[e] = __bfloat16_as_ushort(hb);
        l[e] = __bfloat16_as_ushort(__float2bfloat16_rn(f[e] - __bfloat162float(hb)));
    }
    *reinterpret_cast<uint2 *>(hi + i) = make_uint2((uint32_t)h[0] | ((uint32_t)h[1] << 16), (uint32_t)h[2] | ((uint32_t)h[3] << 16));
    *reinterpret_cast<uint2 *>(lo + i) = make_uint2((uint32_t)l[0] | ((uint32_t)l[1] << 16), (uint32_t)l[2] | ((uint32_t)l[3] << 16));
}
__global__ void __launch_bounds__(PF_THREADS) k_pf_norm_split(const float *x, int n, int norm, const float *gamma, const float *beta,
                                                               float eps, __nv_bfloat16 *hi, __nv_bfloat16 *lo, const float *partial,
                                                               int n_split, int T, const float *bias, float *x_store) {
    pdl_launch_dependents();
    pdl_wait();
    __shared__ float red[2 * PF_THREADS / 32];
    __shared__ float s_pilot;
    const int t = blockIdx.x, tid = threadIdx.x;
    const float *row = x + (size_t)t * n;
    const int n4 = n >> 2;
    if ((n & 3) == 0 && n4 <= PF_VPT * PF_THREADS) {
        // this block's float4 columns: all of the row, or a slice of it (element-wise uses only)
        const int per = (n4 + gridDim.y - 1) / gridDim.y, c_lo = blockIdx.y * per, c_hi = min(n4, c_lo + per);
        float4 v[PF_VPT];
#pragma unroll
        for (int u = 0; u < PF_VPT; ++u) {
            const int i4 = c_lo + tid + u * PF_THREADS;
            v[u] = i4 < c_hi ? __ldcg(reinterpret_cast<const float4 *>(row) + i4) : make_float4(0.f, 0.f, 0.f, 0.f);
        }
        if (n_split > 0) {
#pragma unroll
            for (int u = 0; u < PF_VPT; ++u) {
                const int i4 = c_lo + tid + u * PF_THREADS;
                if (i4 < c_hi && bias) { const float4 b = reinterpret_cast<const float4 *>(bias)[i4]; v[u].x += b.x; v[u].y += b.y; v[u].z += b.z; v[u].w += b.w; }
            }
            for (int z = 0; z < n_split; ++z) {
                float4 p[PF_VPT];
#pragma unroll
                for (int u = 0; u < PF_VPT; ++u) {
                    const int i4 = c_lo + tid + u * PF_THREADS;
                    p[u] = i4 < c_hi ? __ldcg(reinterpret_cast<const float4 *>(partial + ((size_t)z * T + t) * n) + i4) : make_float4(0.f, 0.f, 0.f, 0.f);
                }
#pragma unroll
                for (int u = 0; u < PF_VPT; ++u) { v[u].x += p[u].x; v[u].y += p[u].y; v[u].z += p[u].z; v[u].w += p[u].w; }
            }
#pragma unroll
            for (int u = 0; u < PF_VPT; ++u) {
                const int i4 = c_lo + tid + u * PF_THREADS;
                if (i4 < c_hi) reinterpret_cast<float4 *>(x_store + (size_t)t * n)[i4] = v[u];
            }
        }
        if (!hi) return;
        float mean = 0.f, rstd = 1.f;
        if (gamma) { // (one slice: the block holds the whole row)
            if (tid == 0) s_pilot = norm == NORM_LAYER ? v[0].x : 0.f;
            __syncthreads();
            const float pilot = s_pilot;
            float s1 = 0.f, s2 = 0.f;
#pragma unroll
            for (int u = 0; u < PF_VPT; ++u)
                if (c_lo + tid + u * PF_THREADS < c_hi) {
                    const float a = v[u].x - pilot, b = v[u].y - pilot, c2 = v[u].z - pilot, d2 = v[u].w - pilot;
                    s1 += (a + b) + (c2 + d2);
                    s2 += (a * a + b * b) + (c2 * c2 + d2 * d2);
                }
            s1 = warp_sum(s1);
            s2 = warp_sum(s2);
            if ((tid & 31) == 0) { red[tid >> 5] = s1; red[PF_THREADS / 32 + (tid >> 5)] = s2; }
            __syncthreads();
            s1 = s2 = 0.f;
            for (int w = 0; w < PF_THREADS / 32; ++w) { s1 += red[w]; s2 += red[PF_THREADS / 32 + w]; }
            const float dm = norm == NORM_LAYER ? s1 / (float)n : 0.f;
            mean = pilot + dm;
            rstd = rsqrtf(fmaxf(s2 / (float)n - dm * dm, 0.f) + eps);
        }
#pragma unroll
        for (int u = 0; u < PF_VPT; ++u) {
            const int i4 = c_lo + tid + u * PF_THREADS;
            if (i4 >= c_hi) continue;
            float4 y = v[u];
            if (gamma) {
                const float4 g = reinterpret_cast<const float4 *>(gamma)[i4];
                y.x = (y.x - mean) * rstd * g.x; y.y = (y.y - mean) * rstd * g.y; y.z = (y.z - mean) * rstd * g.z; y.w = (y.w - mean) * rstd * g.w;
                if (beta) { const float4 b = reinterpret_cast<const float4 *>(beta)[i4]; y.x += b.x; y.y += b.y; y.z += b.z; y.w += b.w; }
            }
            pf_split_store4(hi, lo, (size_t)t * n + 4 * (size_t)i4, y);
        }
        return;
    }
    // ---- long or odd rows: plain loops (one slice)
    if (blockIdx.y != 0) return;
    if (n_split > 0) {
        float *dst = x_store + (size_t)t * n;
        for (int i = tid; i < n; i += PF_THREADS) {
            float v = row[i] + (bias ? bias[i] : 0.f);
            for (int z = 0; z < n_split; ++z) v += partial[((size_t)z * T + t) * n + i];
            dst[i] = v;
        }
        row = dst;
        __syncthreads();
    }
    if (!hi) return;
    float mean = 0.f, rstd = 1.f;
    if (gamma) {
        const float pilot = norm == NORM_LAYER ? row[0] : 0.f;
        float s1 = 0.f, s2 = 0.f;
        for (int i = tid; i < n; i += PF_THREADS) { const float c = row[i] - pilot; s1 += c; s2 += c * c; }
        s1 = warp_sum(s1);
        s2 = warp_sum(s2);
        if ((tid & 31) == 0) { red[tid >> 5] = s1; red[PF_THREADS / 32 + (tid >> 5)] = s2; }
        __syncthreads();
        s1 = s2 = 0.f;
        for (int w = 0; w < PF_THREADS / 32; ++w) { s1 += red[w]; s2 += red[PF_THREADS / 32 + w]; }
        const float dm = norm == NORM_LAYER ? s1 / (float)n : 0.f;
        mean = pilot + dm;
        rstd = rsqrtf(fmaxf(s2 / (float)n - dm * dm, 0.f) + eps);
    }
    for (int i = tid; i < n; i += PF_THREADS) {
        float v = row[i];
        if (gamma) { v = (v - mean) * rstd * gamma[i]; if (beta) v += beta[i]; }
        pf_split_store(hi, lo, (size_t)t * n + i, v);
    }
}

// h = SiLU(g) * u, split.  grid (T, column slices)
__global__ void k_pf_swiglu_split(const float *g, const float *u, int n, __nv_bfloat16 *hi, __nv_bfloat16 *lo) {
    pdl_launch_dependents();
    pdl_wait();
    const int t = blockIdx.x;
    for (int i = blockIdx.y * blockDim.x + threadIdx.x; i < n; i += gridDim.y * blockDim.x) {
        const size_t k = (size_t)t * n + i;
        pf_split_store(hi, lo, k, silu_f(g[k]) * u[k]);
    }
}

// qkv[t][q | k | v] (bias already added) -> q[t][:] (rotated) and the cache rows pos0 + t (k rotated).  grid (T)
template <typename KT>
__global__ void k_pf_rope_append(const float *qkv, int q_rows, int kv_rows, int hd, int rope, const float *rope_cos,
                                 const float *rope_sin, KvView kv, int layer_local, const int *pos, int slot, float *q_out) {
    pdl_launch_dependents();
    pdl_wait();
    const int t = blockIdx.x, p = pos[slot] + t, half = hd >> 1, rows = q_rows + 2 * kv_rows;
    const float *src = qkv + (size_t)t * rows;
    for (int r = threadIdx.x; r < rows; r += blockDim.x) {
        float y = src[r];
        if (rope && r < q_rows + kv_rows) {
            const int e = r % hd, i = e % half;
            const float c = rope_cos[(size_t)p * half + i], s = rope_sin[(size_t)p * half + i];
            y = e < half ? y * c - src[r + half] * s : y * c + src[r - half] * s;
        }
        if (r < q_rows) q_out[(size_t)t * q_rows + r] = y;
        else {
            const int rk = r - q_rows, which = rk >= kv_rows, rl = rk - which * kv_rows;
            kv_store<KT>(kv_addr<KT>(kv, slot, layer_local, which, rl / hd, p, rl % hd), y);
        }
    }
}

// Causal attention of the T new positions over the slot's cache (rows 0 .. pos0 + t for position t).
// grid (n_head, T); same row-sharing scheme as k_attn_decode, no sequence split.
template <typename KT, int HD>
__global__ void __launch_bounds__(ATT_THREADS) k_pf_attn(const float *q, __nv_bfloat16 *o_hi, __nv_bfloat16 *o_lo, KvView kv,
                                                          int layer_local, int n_head, const int *pos, int slot, float scale) {
    constexpr int EPL = 16 / sizeof(KT), LPR = HD / EPL, RPW = 32 / LPR, NG = ATT_WARPS * RPW;
    __shared__ float sm_m[NG], sm_l[NG];
    __shared__ float sm_o[NG][HD];
    pdl_launch_dependents();
    pdl_wait();
    const int h = blockIdx.x, t = blockIdx.y, tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int sub = lane % LPR, grp = lane / LPR;
    const int n_keys = pos[slot] + t + 1;
    const int kvh = h / (n_head / kv.n_kv_head);
    float qv[EPL], ov[EPL];
#pragma unroll
    for (int e = 0; e < EPL; ++e) { qv[e] = q[((size_t)t * n_head + h) * HD + sub * EPL + e] * scale; ov[e] = 0.f; }
    float m = -INFINITY, l = 0.f;
    for (int j0 = warp * RPW; j0 < n_keys; j0 += NG) {
        const int j = j0 + grp;
        const bool live = j < n_keys;
        const KT *kp = kv_addr<KT>(kv, slot, layer_local, 0, kvh, live ? j : 0, sub * EPL);
        const KT *vp = kp + (size_t)kv.n_kv_head * kv.page_tokens * HD;
        WVec<KT> kk, vv;
        kk.load(kp);
        vv.load(vp);
        float kf[EPL], vf[EPL];
        kk.unpack(kf);
        vv.unpack(vf);
        float s = 0.f;
#pragma unroll
        for (int e = 0; e < EPL; ++e) s = fmaf(qv[e], kf[e], s);
#pragma unroll
        for (int w = LPR / 2; w > 0; w >>= 1) s += __shfl_xor_sync(0xffffffffu, s, w);
        if (live) {
            const float mn = fmaxf(m, s), corr = expf(m - mn), pr = expf(s - mn);
            l = l * corr + pr;
#pragma unroll
            for (int e = 0; e < EPL; ++e) ov[e] = ov[e] * corr + pr * vf[e];
            m = mn;
        }
    }
    const int g = warp * RPW + grp;
    if (sub == 0) { sm_m[g] = m; sm_l[g] = l; }
#pragma unroll
    for (int e = 0; e < EPL; ++e) sm_o[g][sub * EPL + e] = ov[e];
    __syncthreads();
    if (tid < HD) {
        float M = -INFINITY;
#pragma unroll
        for (int g2 = 0; g2 < NG; ++g2) M = fmaxf(M, sm_m[g2]);
        float L = 0.f, O = 0.f;
#pragma unroll
        for (int g2 = 0; g2 < NG; ++g2) {
            const float w = sm_m[g2] == -INFINITY ? 0.f : expf(sm_m[g2] - M);
            L += sm_l[g2] * w;
            O += sm_o[g2][tid] * w;
        }
        pf_split_store(o_hi, o_lo, ((size_t)t * n_head + h) * HD + tid, O / L);
    }
}

// The same for a batch of items of different slots (a group's decode step): item i sits at pos[slot_i] + off_i.
// grid (n items, row slices)
template <typename KT>
__global__ void k_bt_rope_append(const float *qkv, int q_rows, int kv_rows, int hd, int rope, const float *rope_cos,
                                 const float *rope_sin, KvView kv, int layer_local, const int *pos, Batch bt, float *q_out) {
    pdl_launch_dependents();
    pdl_wait();
    const int t = blockIdx.x, slot = bt.slot[t], p = pos[slot] + bt.off[t], half = hd >> 1, rows = q_rows + 2 * kv_rows;
    const float *src = qkv + (size_t)t * rows;
    for (int r = blockIdx.y * blockDim.x + threadIdx.x; r < rows; r += gridDim.y * blockDim.x) {
        float y = src[r];
        if (rope && r < q_rows + kv_rows) {
            const int e = r % hd, i = e % half;
            const float c = rope_cos[(size_t)p * half + i], s = rope_sin[(size_t)p * half + i];
            y = e < half ? y * c - src[r + half] * s : y * c + src[r - half] * s;
        }
        if (r < q_rows) q_out[(size_t)t * q_rows + r] = y;
        else {
            const int rk = r - q_rows, which = rk >= kv_rows, rl = rk - which * kv_rows;
            kv_store<KT>(kv_addr<KT>(kv, slot, layer_local, which, rl / hd, p, rl % hd), y);
        }
    }
}

__global__ void k_bt_advance(int *pos, Batch bt) {
    pdl_launch_dependents();
    pdl_wait();
    const int i = threadIdx.x;
    if (blockIdx.x == 0 && i < bt.n && bt.adv[i]) pos[bt.slot[i]] += bt.adv[i];
}

__global__ void k_pf_advance(int *pos, int slot, int by) {
    pdl_launch_dependents();
    pdl_wait();
    if (threadIdx.x == 0 && blockIdx.x == 0) pos[slot] += by;
}

} // namespace mdi
