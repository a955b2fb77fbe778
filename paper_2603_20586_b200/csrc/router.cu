// Router gate kernel: lambda = softmax over three levels of (R W_r + b_r), one gate per token
// (Alg. 1 step 12 / Alg. 2 step 5), plus the hard top-1 / top-2 and uniform routing variants
// (Table 10).  HBM-bound: every row of R is read exactly once with 16-byte loads; each warp owns
// four rows at a time so that one read of W_r serves four rows.
// Also the router's backward: dW_r = R^T dG, db_r = sum dG (two deterministic passes).
#include "common.cuh"

namespace mka {
namespace {

constexpr int kRowsPerWarp = 4;
constexpr int kWarps = 8;

__device__ __forceinline__ void finish_row(float g0, float g1, float g2, int route, long long row, float* gate,
                                           float* log2_gate, int8_t* idx) {
    float g[3] = {g0, g1, g2};
    float mx = fmaxf(g0, fmaxf(g1, g2));
    float e[3], sum = 0.f;
#pragma unroll
    for (int l = 0; l < 3; ++l) { e[l] = expf(g[l] - mx); sum += e[l]; }
    float lam[3];
#pragma unroll
    for (int l = 0; l < 3; ++l) lam[l] = e[l] / sum;
    int8_t id0 = -1, id1 = -1;
    if (route == MKA_ROUTE_UNIFORM) {
        lam[0] = lam[1] = lam[2] = 1.0f / 3.0f;
    } else if (route == MKA_ROUTE_TOP1 || route == MKA_ROUTE_TOP2) {
        int keep = route == MKA_ROUTE_TOP1 ? 1 : 2;
        bool kept[3] = {false, false, false};
        for (int k = 0; k < keep; ++k) {            // largest logit first; a tie goes to the lower level
            int best = -1;
#pragma unroll
            for (int l = 0; l < 3; ++l)
                if (!kept[l] && (best < 0 || g[l] > g[best])) best = l;
            kept[best] = true;
        }
        float ks = 0.f;
#pragma unroll
        for (int l = 0; l < 3; ++l) if (kept[l]) ks += lam[l];
#pragma unroll
        for (int l = 0; l < 3; ++l) lam[l] = kept[l] ? lam[l] / ks : 0.f;
#pragma unroll
        for (int l = 0; l < 3; ++l)
            if (kept[l]) { if (id0 < 0) id0 = (int8_t)l; else id1 = (int8_t)l; }
    }
#pragma unroll
    for (int l = 0; l < 3; ++l) {
        gate[row * 3 + l] = lam[l];
        if (log2_gate) log2_gate[row * 3 + l] = lam[l] > 0.f ? log2f(lam[l]) : -INFINITY;
    }
    if (idx) { idx[row * 2] = id0; idx[row * 2 + 1] = id1; }
}

template <typename T> struct Vec8;  // eight consecutive elements as floats
template <> struct Vec8<__nv_bfloat16> {
    static __device__ __forceinline__ void load(const __nv_bfloat16* p, float (&x)[8]) {
        uint4 u = __ldg(reinterpret_cast<const uint4*>(p));
        uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            x[2 * i] = __uint_as_float(w[i] << 16);
            x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
        }
    }
};
template <> struct Vec8<float> {
    static __device__ __forceinline__ void load(const float* p, float (&x)[8]) {
        float4 a = __ldg(reinterpret_cast<const float4*>(p));
        float4 b = __ldg(reinterpret_cast<const float4*>(p) + 1);
        x[0] = a.x; x[1] = a.y; x[2] = a.z; x[3] = a.w; x[4] = b.x; x[5] = b.y; x[6] = b.z; x[7] = b.w;
    }
};

template <typename T, bool VEC>
__global__ void __launch_bounds__(kWarps * 32)
router_kernel(const T* __restrict__ R, const float* __restrict__ W_r, const float* __restrict__ b_r,
              long long rows, int D, int route, float* __restrict__ gate, float* __restrict__ log2_gate,
              int8_t* __restrict__ idx) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const long long row0 = ((long long)blockIdx.x * kWarps + warp) * kRowsPerWarp;
    if (row0 >= rows) return;
    float acc[kRowsPerWarp][3];
#pragma unroll
    for (int r = 0; r < kRowsPerWarp; ++r) acc[r][0] = acc[r][1] = acc[r][2] = 0.f;
    const T* rp[kRowsPerWarp];
#pragma unroll
    for (int r = 0; r < kRowsPerWarp; ++r) {
        long long rr = row0 + r < rows ? row0 + r : rows - 1;   // clamp: tail rows recompute the last row
        rp[r] = R + rr * (long long)D;
    }
    if (VEC) {
        for (int c = lane * 8; c < D; c += 32 * 8) {
            float w[24];
            const float4* wp = reinterpret_cast<const float4*>(W_r + (long long)c * 3);
#pragma unroll
            for (int i = 0; i < 6; ++i) {
                float4 v = __ldg(wp + i);
                w[4 * i] = v.x; w[4 * i + 1] = v.y; w[4 * i + 2] = v.z; w[4 * i + 3] = v.w;
            }
#pragma unroll
            for (int r = 0; r < kRowsPerWarp; ++r) {
                float x[8];
                Vec8<T>::load(rp[r] + c, x);
#pragma unroll
                for (int i = 0; i < 8; ++i) {
                    acc[r][0] = fmaf(x[i], w[3 * i], acc[r][0]);
                    acc[r][1] = fmaf(x[i], w[3 * i + 1], acc[r][1]);
                    acc[r][2] = fmaf(x[i], w[3 * i + 2], acc[r][2]);
                }
            }
        }
    } else {
        for (int c = lane; c < D; c += 32) {
            float w0 = W_r[c * 3], w1 = W_r[c * 3 + 1], w2 = W_r[c * 3 + 2];
#pragma unroll
            for (int r = 0; r < kRowsPerWarp; ++r) {
                float x = Elem<T>::ld(rp[r] + c);
                acc[r][0] = fmaf(x, w0, acc[r][0]);
                acc[r][1] = fmaf(x, w1, acc[r][1]);
                acc[r][2] = fmaf(x, w2, acc[r][2]);
            }
        }
    }
#pragma unroll
    for (int r = 0; r < kRowsPerWarp; ++r)
#pragma unroll
        for (int l = 0; l < 3; ++l) acc[r][l] = warp_sum(acc[r][l]);
    if (lane < kRowsPerWarp && row0 + lane < rows) {
        float g0 = 0.f, g1 = 0.f, g2 = 0.f;
#pragma unroll
        for (int r = 0; r < kRowsPerWarp; ++r)
            if (lane == r) { g0 = acc[r][0]; g1 = acc[r][1]; g2 = acc[r][2]; }
        if (b_r) { g0 += b_r[0]; g1 += b_r[1]; g2 += b_r[2]; }
        finish_row(g0, g1, g2, route, row0 + lane, gate, log2_gate, idx);
    }
}

// dW_r partials: CTA (row chunk, column block); thread = one column of R, loops over the chunk's rows.
template <typename T>
__global__ void __launch_bounds__(256)
router_bwd_partial_kernel(const T* __restrict__ R, const float* __restrict__ dG, long long rows, int D,
                          int n_row_chunks, float* __restrict__ partial) {
    const int c = blockIdx.x * 256 + threadIdx.x;
    const int chunk = blockIdx.y;
    const long long per = (rows + n_row_chunks - 1) / n_row_chunks;
    const long long r0 = chunk * per, r1 = r0 + per < rows ? r0 + per : rows;
    __shared__ float g[64][3];
    float a0 = 0.f, a1 = 0.f, a2 = 0.f;
    for (long long rb = r0; rb < r1; rb += 64) {
        __syncthreads();
        if (threadIdx.x < 64 * 3) {
            long long rr = rb + threadIdx.x / 3;
            g[threadIdx.x / 3][threadIdx.x % 3] = rr < r1 ? dG[rr * 3 + threadIdx.x % 3] : 0.f;
        }
        __syncthreads();
        if (c < D) {
            int lim = (int)((r1 - rb) < 64 ? (r1 - rb) : 64);
            for (int i = 0; i < lim; ++i) {
                float x = Elem<T>::ld(R + (rb + i) * (long long)D + c);
                a0 = fmaf(x, g[i][0], a0); a1 = fmaf(x, g[i][1], a1); a2 = fmaf(x, g[i][2], a2);
            }
        }
    }
    if (c < D) {
        float* o = partial + ((long long)chunk * D + c) * 3;
        o[0] = a0; o[1] = a1; o[2] = a2;
    }
}

// The same with four consecutive columns per thread (one 8- or 16-byte load per row), rows taken four at a time so that
// four loads are in flight; used when D is a multiple of 4 and R is 16-byte aligned.  Per column the rows are added in
// the same order as above.
template <typename T>
__global__ void __launch_bounds__(256)
router_bwd_partial4_kernel(const T* __restrict__ R, const float* __restrict__ dG, long long rows, int D,
                           int n_row_chunks, float* __restrict__ partial) {
    const int c = (blockIdx.x * 256 + threadIdx.x) * 4;
    const int chunk = blockIdx.y;
    const long long per = (rows + n_row_chunks - 1) / n_row_chunks;
    const long long r0 = chunk * per, r1 = r0 + per < rows ? r0 + per : rows;
    __shared__ float g[64][3];
    float a[4][3];
#pragma unroll
    for (int j = 0; j < 4; ++j) a[j][0] = a[j][1] = a[j][2] = 0.f;
    auto load4 = [&](long long r, float (&x)[4]) {
        if (sizeof(T) == 2) {
            const uint2 w = __ldg(reinterpret_cast<const uint2*>(R + r * (long long)D + c));
            x[0] = __uint_as_float(w.x << 16); x[1] = __uint_as_float(w.x & 0xffff0000u);
            x[2] = __uint_as_float(w.y << 16); x[3] = __uint_as_float(w.y & 0xffff0000u);
        } else {
            const float4 w = __ldg(reinterpret_cast<const float4*>(R + r * (long long)D + c));
            x[0] = w.x; x[1] = w.y; x[2] = w.z; x[3] = w.w;
        }
    };
    for (long long rb = r0; rb < r1; rb += 64) {
        __syncthreads();
        if (threadIdx.x < 64 * 3) {
            long long rr = rb + threadIdx.x / 3;
            g[threadIdx.x / 3][threadIdx.x % 3] = rr < r1 ? dG[rr * 3 + threadIdx.x % 3] : 0.f;
        }
        __syncthreads();
        if (c < D) {
            const int lim = (int)((r1 - rb) < 64 ? (r1 - rb) : 64);
            int i = 0;
            for (; i + 4 <= lim; i += 4) {
                float x[4][4];
#pragma unroll
                for (int u = 0; u < 4; ++u) load4(rb + i + u, x[u]);
#pragma unroll
                for (int u = 0; u < 4; ++u)
#pragma unroll
                    for (int j = 0; j < 4; ++j) {
                        a[j][0] = fmaf(x[u][j], g[i + u][0], a[j][0]);
                        a[j][1] = fmaf(x[u][j], g[i + u][1], a[j][1]);
                        a[j][2] = fmaf(x[u][j], g[i + u][2], a[j][2]);
                    }
            }
            for (; i < lim; ++i) {
                float x[4];
                load4(rb + i, x);
#pragma unroll
                for (int j = 0; j < 4; ++j) {
                    a[j][0] = fmaf(x[j], g[i][0], a[j][0]); a[j][1] = fmaf(x[j], g[i][1], a[j][1]); a[j][2] = fmaf(x[j], g[i][2], a[j][2]);
                }
            }
        }
    }
    if (c < D) {
        float* o = partial + ((long long)chunk * D + c) * 3;
#pragma unroll
        for (int j = 0; j < 4; ++j) { o[3 * j] = a[j][0]; o[3 * j + 1] = a[j][1]; o[3 * j + 2] = a[j][2]; }
    }
}

__global__ void router_bwd_reduce_kernel(const float* __restrict__ partial, int D, int n_row_chunks,
                                         float* __restrict__ dW_r) {
    int i = blockIdx.x * blockDim.x + threadIdx.x;   // over D*3
    if (i >= D * 3) return;
    float s = 0.f;
    for (int k = 0; k < n_row_chunks; ++k) s += partial[(long long)k * D * 3 + i];
    dW_r[i] = s;
}

// db_r = sum over rows of dG: one CTA, fixed-order tree.
__global__ void __launch_bounds__(256) router_bias_grad_kernel(const float* __restrict__ dG, long long rows,
                                                               float* __restrict__ db_r) {
    __shared__ float sm[256][3];
    float a[3] = {0.f, 0.f, 0.f};
    for (long long r = threadIdx.x; r < rows; r += 256)
        for (int l = 0; l < 3; ++l) a[l] += dG[r * 3 + l];
    for (int l = 0; l < 3; ++l) sm[threadIdx.x][l] = a[l];
    __syncthreads();
    for (int s = 128; s > 0; s >>= 1) {
        if (threadIdx.x < s)
            for (int l = 0; l < 3; ++l) sm[threadIdx.x][l] += sm[threadIdx.x + s][l];
        __syncthreads();
    }
    if (threadIdx.x < 3) db_r[threadIdx.x] = sm[0][threadIdx.x];
}

}  // namespace

cudaError_t launch_router(const void* R, const float* W_r, const float* b_r, long long rows, int D, int r_dtype,
                          int route, float* gate, float* log2_gate, int8_t* idx, cudaStream_t st) {
    if (rows == 0) return cudaSuccess;
    const long long rows_per_cta = kWarps * kRowsPerWarp;
    dim3 grid((unsigned)((rows + rows_per_cta - 1) / rows_per_cta)), block(kWarps * 32);
    const bool vec = (D % 8 == 0) && ((uintptr_t)R % 16 == 0) && ((uintptr_t)W_r % 16 == 0);
    if (r_dtype == MKA_BF16) {
        auto* p = static_cast<const __nv_bfloat16*>(R);
        if (vec) router_kernel<__nv_bfloat16, true><<<grid, block, 0, st>>>(p, W_r, b_r, rows, D, route, gate, log2_gate, idx);
        else router_kernel<__nv_bfloat16, false><<<grid, block, 0, st>>>(p, W_r, b_r, rows, D, route, gate, log2_gate, idx);
    } else {
        auto* p = static_cast<const float*>(R);
        if (vec) router_kernel<float, true><<<grid, block, 0, st>>>(p, W_r, b_r, rows, D, route, gate, log2_gate, idx);
        else router_kernel<float, false><<<grid, block, 0, st>>>(p, W_r, b_r, rows, D, route, gate, log2_gate, idx);
    }
    return cudaGetLastError();
}

cudaError_t launch_router_bwd(const void* R, int r_dtype, const float* dG, long long rows, int D, float* dW_r,
                              float* db_r, float* partial, int n_row_chunks, cudaStream_t st) {
    if (dW_r && D % 4 == 0 && (reinterpret_cast<uintptr_t>(R) & 15) == 0) {
        dim3 grid((D / 4 + 255) / 256, n_row_chunks), block(256);
        if (r_dtype == MKA_BF16)
            router_bwd_partial4_kernel<__nv_bfloat16><<<grid, block, 0, st>>>(static_cast<const __nv_bfloat16*>(R), dG, rows, D, n_row_chunks, partial);
        else
            router_bwd_partial4_kernel<float><<<grid, block, 0, st>>>(static_cast<const float*>(R), dG, rows, D, n_row_chunks, partial);
        router_bwd_reduce_kernel<<<(D * 3 + 255) / 256, 256, 0, st>>>(partial, D, n_row_chunks, dW_r);
    } else if (dW_r) {
        dim3 grid((D + 255) / 256, n_row_chunks), block(256);
        if (r_dtype == MKA_BF16)
            router_bwd_partial_kernel<__nv_bfloat16><<<grid, block, 0, st>>>(static_cast<const __nv_bfloat16*>(R), dG, rows, D, n_row_chunks, partial);
        else
            router_bwd_partial_kernel<float><<<grid, block, 0, st>>>(static_cast<const float*>(R), dG, rows, D, n_row_chunks, partial);
        router_bwd_reduce_kernel<<<(D * 3 + 255) / 256, 256, 0, st>>>(partial, D, n_row_chunks, dW_r);
    }
    if (db_r) router_bias_grad_kernel<<<1, 256, 0, st>>>(dG, rows, db_r);
    return cudaGetLastError();
}

}  // namespace mka
