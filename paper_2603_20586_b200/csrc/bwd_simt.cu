// CUDA-core backward of Eq. 5 (derived by differentiating it; the paper prints no backward).
// With p = lambda exp(s - LSE) on the visible set, D_t = dO_t . O_t and dS = p (dO_t . v - D_t):
//   kernel delta : D[b,h,t]
//   kernel dq    : dQ_t = tau sum_{l,j} dS k_{l,j};  per-head gate-logit gradient G[b,h,t,l] = sum_j dS
//   kernel dkv   : dK_{l,j} = tau sum_t dS q_t;  dV_{l,j} = sum_t p dO_t       (one launch per level)
//   kernel dgate : dG[b,t,l] = sum_h G[b,h,t,l]                               (fixed order)
// Every output element is produced by exactly one thread in a fixed summation order, so the result is
// deterministic.  fp32 arithmetic; tiles of 32 x 32 (query x key) staged in shared memory.
#include "common.cuh"

namespace mka {
namespace {

constexpr int kRows = 32, kKeys = 32, kWarpRows = 4, kThreads = 256;

template <typename T, int DH>
__global__ void __launch_bounds__(256) bwd_delta_kernel(const T* __restrict__ O, const T* __restrict__ dO,
                                                        long long rows, float* __restrict__ delta) {
    const int lane = threadIdx.x & 31;
    const long long row = (long long)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (row >= rows) return;
    float s = 0.f;
    for (int c = lane; c < DH; c += 32) s = fmaf(Elem<T>::ld(O + row * DH + c), Elem<T>::ld(dO + row * DH + c), s);
    s = warp_sum(s);
    if (lane == 0) delta[row] = s;
}

template <typename T, int DH>
__global__ void __launch_bounds__(kThreads) bwd_dq_kernel(const BwdParams p) {
    constexpr int CPL = (DH + 31) / 32, LD = DH + 1;
    extern __shared__ float smem[];
    float* qs = smem;                 // [kRows][DH]  tau * q
    float* gs = qs + kRows * DH;      // [kRows][DH]  dO
    float* ks = gs + kRows * DH;      // [kKeys][LD]
    float* vs = ks + kKeys * LD;      // [kKeys][LD]
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int b = blockIdx.z, h = blockIdx.y;
    const long long t0 = (long long)blockIdx.x * kRows;
    const long long bh = (long long)b * p.H + h;
    const T* Q = static_cast<const T*>(p.Q) + bh * p.T * DH;
    const T* dO = static_cast<const T*>(p.dO) + bh * p.T * DH;
    for (int i = threadIdx.x; i < kRows * DH; i += kThreads) {
        long long t = t0 + i / DH;
        qs[i] = t < p.T ? Elem<T>::ld(Q + t * DH + (i % DH)) * p.scale : 0.f;
        gs[i] = t < p.T ? Elem<T>::ld(dO + t * DH + (i % DH)) : 0.f;
    }
    float lse[kWarpRows], dlt[kWarpRows], acc[kWarpRows][CPL];
    float Ap[kWarpRows][3], Sp[kWarpRows][3];   // per level: sum_j p dP and sum_j p (for the gate gradient)
#pragma unroll
    for (int r = 0; r < kWarpRows; ++r) {
        long long t = t0 + warp * kWarpRows + r;
        long long tc = t < p.T ? t : p.T - 1;
        lse[r] = p.LSE[bh * p.T + tc];
        dlt[r] = p.delta[bh * p.T + tc];
#pragma unroll
        for (int k = 0; k < CPL; ++k) acc[r][k] = 0.f;
        Ap[r][0] = Ap[r][1] = Ap[r][2] = 0.f;
        Sp[r][0] = Sp[r][1] = Sp[r][2] = 0.f;
    }
    const long long t_last = (t0 + kRows - 1 < p.T ? t0 + kRows - 1 : p.T - 1);
#pragma unroll
    for (int lvl = 0; lvl < 3; ++lvl) {
        const LevelDev L = p.L[lvl];
        if (L.n == 0) continue;
        long long lo_f, hi_f, lo_l, hi_l;
        visible_range(lvl, t0 + p.q_offset, p.window, L.n, 0, lo_f, hi_f);
        visible_range(lvl, t_last + p.q_offset, p.window, L.n, 0, lo_l, hi_l);
        const long long lo = lo_f, hi = hi_l > hi_f ? hi_l : hi_f;
        const T* Kp = static_cast<const T*>(L.k) + b * L.sb + (h / p.kv_group) * L.sh;
        const T* Vp = static_cast<const T*>(L.v) + b * L.sb + (h / p.kv_group) * L.sh;
        float lam[kWarpRows];
        long long rlo[kWarpRows], rhi[kWarpRows];
#pragma unroll
        for (int r = 0; r < kWarpRows; ++r) {
            long long t = t0 + warp * kWarpRows + r;
            long long tc = t < p.T ? t : p.T - 1;
            lam[r] = p.gate[((long long)b * p.T + tc) * 3 + lvl];
            visible_range(lvl, tc + p.q_offset, p.window, L.n, 0, rlo[r], rhi[r]);
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
            float s[kWarpRows], dp[kWarpRows];
#pragma unroll
            for (int r = 0; r < kWarpRows; ++r) s[r] = dp[r] = 0.f;
            const float* kr = ks + lane * LD;
            const float* vr = vs + lane * LD;
            const float* qw = qs + warp * kWarpRows * DH;
            const float* gw = gs + warp * kWarpRows * DH;
#pragma unroll 4
            for (int c = 0; c < DH; ++c) {
                float kv = kr[c], vv = vr[c];
#pragma unroll
                for (int r = 0; r < kWarpRows; ++r) {
                    s[r] = fmaf(qw[r * DH + c], kv, s[r]);
                    dp[r] = fmaf(gw[r * DH + c], vv, dp[r]);
                }
            }
            const long long j = j0 + lane;
            float ds[kWarpRows];
#pragma unroll
            for (int r = 0; r < kWarpRows; ++r) {
                const bool vis = (j >= rlo[r]) && (j < rhi[r]) && lam[r] > 0.f;
                const float pr = vis ? lam[r] * expf(s[r] - lse[r]) : 0.f;
                ds[r] = pr * (dp[r] - dlt[r]);
                Ap[r][lvl] = fmaf(pr, dp[r], Ap[r][lvl]);
                Sp[r][lvl] += pr;
            }
#pragma unroll 4
            for (int jj = 0; jj < kKeys; ++jj) {
                float dj[kWarpRows];
#pragma unroll
                for (int r = 0; r < kWarpRows; ++r) dj[r] = __shfl_sync(0xffffffffu, ds[r], jj);
#pragma unroll
                for (int k = 0; k < CPL; ++k) {
                    int c = lane + 32 * k;
                    float kv = c < DH ? ks[jj * LD + c] : 0.f;
#pragma unroll
                    for (int r = 0; r < kWarpRows; ++r) acc[r][k] = fmaf(dj[r], kv, acc[r][k]);
                }
            }
        }
    }
    T* dQ = static_cast<T*>(p.dQ) + bh * p.T * DH;
#pragma unroll
    for (int r = 0; r < kWarpRows; ++r) {
        long long t = t0 + warp * kWarpRows + r;
        if (t >= p.T) continue;
#pragma unroll
        for (int k = 0; k < CPL; ++k) {
            int c = lane + 32 * k;
            if (c < DH) Elem<T>::st(dQ + t * DH + c, acc[r][k] * p.scale);
        }
        // Gate-logit gradient G_l = sum_{j in l} p (dP - D).  Here D is taken as sum_{l,j} p dP / sum p, which
        // equals dO.O exactly in real arithmetic but does not inherit the rounding of O to its storage
        // type, so that sum_l G_l = 0 holds to fp32 accuracy.
        float a[3], sp[3];
#pragma unroll
        for (int l = 0; l < 3; ++l) { a[l] = warp_sum(Ap[r][l]); sp[l] = warp_sum(Sp[r][l]); }
        const float stot = sp[0] + sp[1] + sp[2];
        const float dd = stot > 0.f ? (a[0] + a[1] + a[2]) / stot : 0.f;
#pragma unroll
        for (int l = 0; l < 3; ++l)
            if (lane == 0) p.Gpart[(bh * p.T + t) * 3 + l] = a[l] - sp[l] * dd;
    }
}

// One CTA = 32 key rows of one level of one (batch, head); loops over the query tiles that see them.
template <typename T, int DH>
__global__ void __launch_bounds__(kThreads) bwd_dkv_kernel(const BwdParams p, const int lvl) {
    constexpr int CPL = (DH + 31) / 32, LD = DH + 1;
    extern __shared__ float smem[];
    float* ksm = smem;                // [kKeys][DH]  tau * k   (this CTA's key rows)
    float* vsm = ksm + kKeys * DH;    // [kKeys][DH]
    float* qs = vsm + kKeys * DH;     // [kRows][LD]  query tile
    float* gs = qs + kRows * LD;      // [kRows][LD]  dO tile
    __shared__ float s_lse[kRows], s_dlt[kRows], s_lam[kRows];
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int b = blockIdx.z, h = blockIdx.y;               // h: KV head; its query heads h * G .. h * G + G - 1 are summed
    const LevelDev L = p.L[lvl];
    const LevelGradDev dL = p.dL[lvl];
    const long long j0 = (long long)blockIdx.x * kKeys;
    const T* Kp = static_cast<const T*>(L.k) + b * L.sb + h * L.sh;
    const T* Vp = static_cast<const T*>(L.v) + b * L.sb + h * L.sh;
    for (int i = threadIdx.x; i < kKeys * DH; i += kThreads) {
        long long j = j0 + i / DH;
        ksm[i] = j < L.n ? Elem<T>::ld(Kp + j * L.sn + (i % DH)) * p.scale : 0.f;
        vsm[i] = j < L.n ? Elem<T>::ld(Vp + j * L.sn + (i % DH)) : 0.f;
    }
    float accK[kWarpRows][CPL], accV[kWarpRows][CPL];
#pragma unroll
    for (int r = 0; r < kWarpRows; ++r)
#pragma unroll
        for (int k = 0; k < CPL; ++k) accK[r][k] = accV[r][k] = 0.f;
    // queries that can see any of this CTA's keys: positions p = t + q_offset with
    //   L1: j <= p <= j + W - 1   L2: p >= j   L3: all
    const long long j_last = (j0 + kKeys - 1 < L.n ? j0 + kKeys - 1 : L.n - 1);
    long long t_lo = 0, t_hi = p.T;
    if (lvl == 0) { t_lo = j0 - p.q_offset; t_hi = j_last + p.window - p.q_offset; }
    else if (lvl == 1) { t_lo = j0 - p.q_offset; }
    if (t_lo < 0) t_lo = 0;
    if (t_hi > p.T) t_hi = p.T;
    for (int gq = 0; gq < p.kv_group; ++gq) {
    const long long bh = (long long)b * p.H + (long long)h * p.kv_group + gq;
    const T* Q = static_cast<const T*>(p.Q) + bh * p.T * DH;
    const T* dO = static_cast<const T*>(p.dO) + bh * p.T * DH;
    for (long long tt = (t_lo / kRows) * kRows; tt < t_hi; tt += kRows) {
        __syncthreads();
        for (int i = threadIdx.x; i < kRows * DH; i += kThreads) {
            int r = i / DH, c = i % DH;
            long long t = tt + r;
            qs[r * LD + c] = t < p.T ? Elem<T>::ld(Q + t * DH + c) : 0.f;
            gs[r * LD + c] = t < p.T ? Elem<T>::ld(dO + t * DH + c) : 0.f;
        }
        if (threadIdx.x < kRows) {
            long long t = tt + threadIdx.x;
            bool ok = t < p.T;
            s_lse[threadIdx.x] = ok ? p.LSE[bh * p.T + t] : 0.f;
            s_dlt[threadIdx.x] = ok ? p.delta[bh * p.T + t] : 0.f;
            s_lam[threadIdx.x] = ok ? p.gate[((long long)b * p.T + t) * 3 + lvl] : 0.f;
        }
        __syncthreads();
        // lane = query of the tile; warp rows = keys
        const long long t = tt + lane;
        long long vlo, vhi;
        visible_range(lvl, t + p.q_offset, p.window, L.n, 0, vlo, vhi);
        if (t >= p.T) vhi = vlo;
        const float lam = s_lam[lane], lse = s_lse[lane], dlt = s_dlt[lane];
        float s[kWarpRows], dp[kWarpRows];
#pragma unroll
        for (int r = 0; r < kWarpRows; ++r) s[r] = dp[r] = 0.f;
        const float* qr = qs + lane * LD;
        const float* gr = gs + lane * LD;
        const float* kw = ksm + warp * kWarpRows * DH;
        const float* vw = vsm + warp * kWarpRows * DH;
#pragma unroll 4
        for (int c = 0; c < DH; ++c) {
            float qv = qr[c], gv = gr[c];
#pragma unroll
            for (int r = 0; r < kWarpRows; ++r) {
                s[r] = fmaf(kw[r * DH + c], qv, s[r]);
                dp[r] = fmaf(vw[r * DH + c], gv, dp[r]);
            }
        }
        float pr[kWarpRows], ds[kWarpRows];
#pragma unroll
        for (int r = 0; r < kWarpRows; ++r) {
            const long long j = j0 + warp * kWarpRows + r;
            const bool vis = (j >= vlo) && (j < vhi) && lam > 0.f;
            pr[r] = vis ? lam * expf(s[r] - lse) : 0.f;
            ds[r] = pr[r] * (dp[r] - dlt);
        }
#pragma unroll 4
        for (int q = 0; q < kRows; ++q) {
            float pj[kWarpRows], dj[kWarpRows];
#pragma unroll
            for (int r = 0; r < kWarpRows; ++r) {
                pj[r] = __shfl_sync(0xffffffffu, pr[r], q);
                dj[r] = __shfl_sync(0xffffffffu, ds[r], q);
            }
#pragma unroll
            for (int k = 0; k < CPL; ++k) {
                int c = lane + 32 * k;
                float qv = c < DH ? qs[q * LD + c] : 0.f;
                float gv = c < DH ? gs[q * LD + c] : 0.f;
#pragma unroll
                for (int r = 0; r < kWarpRows; ++r) {
                    accK[r][k] = fmaf(dj[r], qv, accK[r][k]);
                    accV[r][k] = fmaf(pj[r], gv, accV[r][k]);
                }
            }
        }
    }
    }   // query heads of the group
    T* dKp = static_cast<T*>(dL.dk) + b * dL.sb + h * dL.sh;
    T* dVp = static_cast<T*>(dL.dv) + b * dL.sb + h * dL.sh;
#pragma unroll
    for (int r = 0; r < kWarpRows; ++r) {
        long long j = j0 + warp * kWarpRows + r;
        if (j >= L.n) continue;
#pragma unroll
        for (int k = 0; k < CPL; ++k) {
            int c = lane + 32 * k;
            if (c < DH) {
                Elem<T>::st(dKp + j * dL.sn + c, accK[r][k] * p.scale);
                Elem<T>::st(dVp + j * dL.sn + c, accV[r][k]);
            }
        }
    }
}

__global__ void bwd_dgate_kernel(const float* __restrict__ Gpart, int B, int H, long long T, float* __restrict__ dG) {
    long long i = (long long)blockIdx.x * blockDim.x + threadIdx.x;   // over B*T*3
    if (i >= (long long)B * T * 3) return;
    long long b = i / (T * 3), rem = i % (T * 3);
    float s = 0.f;
    for (int h = 0; h < H; ++h) s += Gpart[((b * H + h) * T) * 3 + rem];
    dG[i] = s;
}

}  // namespace

cudaError_t launch_bwd_dgate(const float* Gpart, int B, int H, long long T, float* dG, cudaStream_t st) {
    const long long n = (long long)B * T * 3;
    if (n == 0) return cudaSuccess;
    bwd_dgate_kernel<<<(unsigned)((n + 255) / 256), 256, 0, st>>>(Gpart, B, H, T, dG);
    return cudaGetLastError();
}

namespace {

template <typename T, int DH>
cudaError_t launch_t(const BwdParams& p, cudaStream_t st) {
    const long long rows = (long long)p.B * p.H * p.T;
    cudaError_t e;
    bwd_delta_kernel<T, DH><<<(unsigned)((rows + 7) / 8), 256, 0, st>>>(static_cast<const T*>(p.O), static_cast<const T*>(p.dO), rows, p.delta);
    if ((e = cudaGetLastError()) != cudaSuccess) return e;
    {
        size_t smem = sizeof(float) * (2 * kRows * DH + 2 * kKeys * (DH + 1));
        e = cudaFuncSetAttribute(bwd_dq_kernel<T, DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        dim3 grid((p.T + kRows - 1) / kRows, p.H, p.B);
        bwd_dq_kernel<T, DH><<<grid, kThreads, smem, st>>>(p);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    {
        size_t smem = sizeof(float) * (2 * kKeys * DH + 2 * kRows * (DH + 1));
        e = cudaFuncSetAttribute(bwd_dkv_kernel<T, DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
        if (e != cudaSuccess) return e;
        for (int lvl = 0; lvl < 3; ++lvl) {
            if (p.L[lvl].n == 0) continue;
            dim3 grid((unsigned)((p.L[lvl].n + kKeys - 1) / kKeys), p.H / (p.kv_group > 0 ? p.kv_group : 1), p.B);
            bwd_dkv_kernel<T, DH><<<grid, kThreads, smem, st>>>(p, lvl);
            if ((e = cudaGetLastError()) != cudaSuccess) return e;
        }
    }
    return launch_bwd_dgate(p.Gpart, p.B, p.H, p.T, p.dG, st);
}

template <typename T>
cudaError_t launch_d(const BwdParams& p, cudaStream_t st) {
    switch (p.d) {
        case 32: return launch_t<T, 32>(p, st);
        case 64: return launch_t<T, 64>(p, st);
        case 96: return launch_t<T, 96>(p, st);
        case 128: return launch_t<T, 128>(p, st);
        default: return cudaErrorNotSupported;
    }
}

}  // namespace

cudaError_t launch_bwd_simt(const BwdParams& p, int dtype, cudaStream_t st) {
    if (p.B == 0 || p.H == 0 || p.T == 0) return cudaSuccess;
    return dtype == MKA_BF16 ? launch_d<__nv_bfloat16>(p, st) : launch_d<float>(p, st);
}

}  // namespace mka
