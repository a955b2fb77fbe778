// CUDA-core forward of the gated three-level attention operator.
//   MKA_MODE_FAST: Eq. 5 -- exp(score) weighted by the level's gate, one running (max, sum, acc)
//                  state carried across all three levels (the max shift of Eq. 11-14, key blocks of
//                  32 rows as in Alg. 3, rescale of Eq. 13-14 applied on every block).
//   MKA_MODE_FULL: Alg. 1 -- one softmax state per level, outputs mixed by the gate at the end.
// fp32 arithmetic throughout, so this is the kernel for fp32 problems (tolerance 1e-4) and the
// on-GPU cross-check of the tensor-core kernel.  One CTA = 32 query rows of one (batch, head); each of
// its 8 warps owns 4 rows; a key tile of 32 rows is staged in shared memory as fp32 and each lane
// scores one key of the tile.
#include "common.cuh"

namespace mka {
namespace {

constexpr int kRows = 32;        // query rows per CTA
constexpr int kKeys = 32;        // key rows per shared-memory tile
constexpr int kWarpRows = 4;
constexpr int kThreads = 256;

template <typename T, int DH, int MODE>
__global__ void __launch_bounds__(kThreads) fwd_simt_kernel(const FwdParams p) {
    constexpr int NS = MODE == MKA_MODE_FULL ? 3 : 1;    // softmax states
    constexpr int CPL = (DH + 31) / 32;                  // output columns per lane
    constexpr int LD = DH + 1;                           // padded row pitch (floats)
    extern __shared__ float smem[];
    float* qs = smem;                    // [kRows][DH]
    float* ks = qs + kRows * DH;         // [kKeys][LD]
    float* vs = ks + kKeys * LD;         // [kKeys][LD]

    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int b = blockIdx.z, h = blockIdx.y;
    const long long t0 = (long long)blockIdx.x * kRows;
    const T* Q = static_cast<const T*>(p.Q) + (((long long)b * p.H + h) * p.T) * DH;
    T* O = static_cast<T*>(p.O) + (((long long)b * p.H + h) * p.T) * DH;

    for (int i = threadIdx.x; i < kRows * DH; i += kThreads) {
        long long t = t0 + i / DH;
        qs[i] = t < p.T ? Elem<T>::ld(Q + t * DH + (i % DH)) * p.scale : 0.f;   // tau folded into q
    }

    float m[NS][kWarpRows], z[NS][kWarpRows], acc[NS][kWarpRows][CPL];
#pragma unroll
    for (int s = 0; s < NS; ++s)
#pragma unroll
        for (int r = 0; r < kWarpRows; ++r) {
            m[s][r] = -INFINITY; z[s][r] = 0.f;
#pragma unroll
            for (int k = 0; k < CPL; ++k) acc[s][r][k] = 0.f;
        }

    const long long t_last = (t0 + kRows - 1 < p.T ? t0 + kRows - 1 : p.T - 1);
#pragma unroll
    for (int lvl = 0; lvl < 3; ++lvl) {
        const int st = MODE == MKA_MODE_FULL ? lvl : 0;
        const LevelDev L = p.L[lvl];
        if (L.n == 0) continue;
        // union of the visible ranges of this CTA's rows
        long long lo_first, hi_first, lo_last, hi_last;
        visible_range(lvl, t0 + p.q_offset, p.window, L.n, p.decode, lo_first, hi_first);
        visible_range(lvl, t_last + p.q_offset, p.window, L.n, p.decode, lo_last, hi_last);
        const long long lo = lo_first, hi = hi_last > hi_first ? hi_last : hi_first;
        const T* Kp = static_cast<const T*>(L.k) + b * L.sb + (h / p.kv_group) * L.sh;
        const T* Vp = static_cast<const T*>(L.v) + b * L.sb + (h / p.kv_group) * L.sh;
        float lam[kWarpRows];
        long long rlo[kWarpRows], rhi[kWarpRows];
#pragma unroll
        for (int r = 0; r < kWarpRows; ++r) {
            long long t = t0 + warp * kWarpRows + r;
            long long tc = t < p.T ? t : p.T - 1;
            lam[r] = p.gate[((long long)b * p.T + tc) * 3 + lvl];
            visible_range(lvl, tc + p.q_offset, p.window, L.n, p.decode, rlo[r], rhi[r]);
            if (t >= p.T) rhi[r] = rlo[r];
        }
        for (long long j0 = (lo / kKeys) * kKeys; j0 < hi; j0 += kKeys) {
            __syncthreads();
            for (int i = threadIdx.x; i < kKeys * DH; i += kThreads) {
                int jr = i / DH, c = i % DH;
                long long j = j0 + jr;
                float kv = 0.f, vv = 0.f;
                if (j < L.n) { kv = Elem<T>::ld(Kp + j * L.sn + c); vv = Elem<T>::ld(Vp + j * L.sn + c); }
                ks[jr * LD + c] = kv;
                vs[jr * LD + c] = vv;
            }
            __syncthreads();
            float s[kWarpRows];
#pragma unroll
            for (int r = 0; r < kWarpRows; ++r) s[r] = 0.f;
            const float* kr = ks + lane * LD;
            const float* qw = qs + warp * kWarpRows * DH;
#pragma unroll 8
            for (int c = 0; c < DH; ++c) {
                float kv = kr[c];
#pragma unroll
                for (int r = 0; r < kWarpRows; ++r) s[r] = fmaf(qw[r * DH + c], kv, s[r]);
            }
            const long long j = j0 + lane;
            float pw[kWarpRows];
#pragma unroll
            for (int r = 0; r < kWarpRows; ++r) {
                const bool vis = (j >= rlo[r]) && (j < rhi[r]) && (MODE == MKA_MODE_FULL || lam[r] > 0.f);
                float x = vis ? s[r] : -INFINITY;
                float mx = warp_max(x);
                float m_new = fmaxf(m[st][r], mx);
                float e = (m_new == -INFINITY) ? 0.f : expf(x - m_new);   // masked: exp(-inf) = 0
                float resc = (m[st][r] == -INFINITY) ? 0.f : expf(m[st][r] - m_new);
                if (MODE == MKA_MODE_FAST) e *= lam[r];
                z[st][r] = z[st][r] * resc + warp_sum(e);
#pragma unroll
                for (int k = 0; k < CPL; ++k) acc[st][r][k] *= resc;
                m[st][r] = m_new;
                pw[r] = e;
            }
#pragma unroll 4
            for (int jj = 0; jj < kKeys; ++jj) {
                float pj[kWarpRows];
#pragma unroll
                for (int r = 0; r < kWarpRows; ++r) pj[r] = __shfl_sync(0xffffffffu, pw[r], jj);
#pragma unroll
                for (int k = 0; k < CPL; ++k) {
                    int c = lane + 32 * k;
                    float vv = c < DH ? vs[jj * LD + c] : 0.f;
#pragma unroll
                    for (int r = 0; r < kWarpRows; ++r) acc[st][r][k] = fmaf(pj[r], vv, acc[st][r][k]);
                }
            }
        }
    }

#pragma unroll
    for (int r = 0; r < kWarpRows; ++r) {
        long long t = t0 + warp * kWarpRows + r;
        if (t >= p.T) continue;
        float out[CPL];
#pragma unroll
        for (int k = 0; k < CPL; ++k) out[k] = 0.f;
        if (MODE == MKA_MODE_FAST) {
            float inv = z[0][r] > 0.f ? 1.f / z[0][r] : 0.f;
#pragma unroll
            for (int k = 0; k < CPL; ++k) out[k] = acc[0][r][k] * inv;
            if (p.LSE && lane == 0)
                p.LSE[((long long)b * p.H + h) * p.T + t] = z[0][r] > 0.f ? m[0][r] + logf(z[0][r]) : -INFINITY;
        } else {
#pragma unroll
            for (int s = 0; s < NS; ++s) {
                float lam = p.gate[((long long)b * p.T + t) * 3 + s];
                float w = z[s][r] > 0.f ? lam / z[s][r] : 0.f;
#pragma unroll
                for (int k = 0; k < CPL; ++k) out[k] = fmaf(acc[s][r][k], w, out[k]);
            }
        }
#pragma unroll
        for (int k = 0; k < CPL; ++k) {
            int c = lane + 32 * k;
            if (c < DH) Elem<T>::st(O + t * DH + c, out[k]);
        }
    }
}

template <typename T, int DH>
cudaError_t launch_t(const FwdParams& p, cudaStream_t st) {
    dim3 grid((p.T + kRows - 1) / kRows, p.H, p.B), block(kThreads);
    size_t smem = sizeof(float) * (kRows * DH + 2 * kKeys * (DH + 1));
    cudaError_t e;
    if (p.mode == MKA_MODE_FULL) {
        e = cudaFuncSetAttribute(fwd_simt_kernel<T, DH, MKA_MODE_FULL>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        fwd_simt_kernel<T, DH, MKA_MODE_FULL><<<grid, block, smem, st>>>(p);
    } else {
        e = cudaFuncSetAttribute(fwd_simt_kernel<T, DH, MKA_MODE_FAST>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        fwd_simt_kernel<T, DH, MKA_MODE_FAST><<<grid, block, smem, st>>>(p);
    }
    return cudaGetLastError();
}

template <typename T>
cudaError_t launch_d(const FwdParams& p, cudaStream_t st) {
    switch (p.d) {
        case 32: return launch_t<T, 32>(p, st);
        case 64: return launch_t<T, 64>(p, st);
        case 96: return launch_t<T, 96>(p, st);
        case 128: return launch_t<T, 128>(p, st);
        default: return cudaErrorNotSupported;
    }
}

}  // namespace

cudaError_t launch_fwd_simt(const FwdParams& p, int dtype, cudaStream_t st) {
    if (p.B == 0 || p.H == 0 || p.T == 0) return cudaSuccess;
    return dtype == MKA_BF16 ? launch_d<__nv_bfloat16>(p, st) : launch_d<float>(p, st);
}

}  // namespace mka
