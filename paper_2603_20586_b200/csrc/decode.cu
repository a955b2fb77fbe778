// Split-KV single-token decode of Eq. 5 (all cached rows of the three levels visible).
//
// Kernel 1 (HBM-bound, streams K and V exactly once): grid = (batch*head) x chunks of the split
// table.  A row of d bf16 values is covered by d/8 lanes with one 16-byte load each, so a warp reads
// 32*16 contiguous bytes per instruction; each lane group keeps its own running (max, sum, acc) in the
// base-2 domain (the max shift of Eq. 11-14) and the groups, then the CTA's warps, are merged with
// warp shuffles / shared memory into one UN-GATED partial per chunk: (m_c, z_c, acc_c[d]).
// Kernel 2: per (batch, head), gate-weighted log-sum-exp combine over all chunks of all levels:
//   O = sum_c lam_{l(c)} 2^{m_c-M} acc_c / sum_c lam_{l(c)} 2^{m_c-M} z_c.
#include <mutex>

#include "common.cuh"

namespace mka {
namespace {

constexpr int kWarps = 8;
constexpr int kUnroll = 8;   // independent 16-byte loads in flight per lane, per stream (K and V)

__device__ __forceinline__ uint4 ld_stream(const void* p) {
    uint4 r;
    asm volatile("ld.global.nc.L1::no_allocate.L2::128B.v4.u32 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r.x), "=r"(r.y), "=r"(r.z), "=r"(r.w) : "l"(p));
    return r;
}

__device__ __forceinline__ void unpack8(const uint4& u, float (&x)[8]) {
    const uint32_t w[4] = {u.x, u.y, u.z, u.w};
#pragma unroll
    for (int i = 0; i < 4; ++i) {
        x[2 * i] = __uint_as_float(w[i] << 16);
        x[2 * i + 1] = __uint_as_float(w[i] & 0xffff0000u);
    }
}

template <int DH>
__global__ void __launch_bounds__(kWarps * 32, 2) decode_partial_kernel(const DecodeParams p) {
    constexpr int LPR = DH / 8;          // lanes per row
    constexpr int RPI = 32 / LPR;        // rows per warp-wide load instruction
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int sub = lane % LPR;          // which 8-column slice of the row this lane holds
    const int grp = lane / LPR;          // which row of the instruction
    const long long bh = blockIdx.x / p.total_chunks;
    long long chunk = blockIdx.x % p.total_chunks;
    int lvl = 0;
    while (lvl < 2 && chunk >= p.n_chunks[lvl]) { chunk -= p.n_chunks[lvl]; ++lvl; }
    const LevelDev L = p.L[lvl];
    const int b = (int)(bh / p.H), h = (int)(bh % p.H);
    const long long r_begin = chunk * p.chunk_rows;
    const long long r_end = r_begin + p.chunk_rows < L.n ? r_begin + p.chunk_rows : L.n;
    if (p.gate[b * 3 + lvl] == 0.f) {                  // hard routing switched this level off: do not read it
        float* out = p.partial + (long long)blockIdx.x * (DH + 2);
        for (int i = threadIdx.x; i < DH + 2; i += kWarps * 32) out[i] = i == 0 ? -INFINITY : 0.f;
        return;
    }
    const __nv_bfloat16* Kp = static_cast<const __nv_bfloat16*>(L.k) + b * L.sb + (h / p.kv_group) * L.sh + sub * 8;
    const __nv_bfloat16* Vp = static_cast<const __nv_bfloat16*>(L.v) + b * L.sb + (h / p.kv_group) * L.sh + sub * 8;

    float q[8];
    {
        uint4 u = *reinterpret_cast<const uint4*>(static_cast<const __nv_bfloat16*>(p.q) + bh * DH + sub * 8);
        unpack8(u, q);
        const float c = p.scale * kLog2e;     // scores in the base-2 domain
#pragma unroll
        for (int i = 0; i < 8; ++i) q[i] *= c;
    }
    float m = -INFINITY, z = 0.f, acc[8];
#pragma unroll
    for (int i = 0; i < 8; ++i) acc[i] = 0.f;

    // rows of this chunk are dealt to warps in slabs of RPI*kUnroll consecutive rows
    constexpr int SLAB = RPI * kUnroll;
    for (long long r0 = r_begin + (long long)warp * SLAB; r0 < r_end; r0 += (long long)kWarps * SLAB) {
        uint4 kk[kUnroll], vv[kUnroll];
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            long long r = r0 + u * RPI + grp;
            long long rc = r < r_end ? r : r_end - 1;        // clamp: a tail lane re-reads the last row
            kk[u] = ld_stream(Kp + rc * L.sn);
        }
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            long long r = r0 + u * RPI + grp;
            long long rc = r < r_end ? r : r_end - 1;
            vv[u] = ld_stream(Vp + rc * L.sn);
        }
        float s[kUnroll];
        float smax = -INFINITY;
#pragma unroll
        for (int u = 0; u < kUnroll; ++u) {
            float x[8];
            unpack8(kk[u], x);
            float d0 = 0.f;
#pragma unroll
            for (int i = 0; i < 8; ++i) d0 = fmaf(q[i], x[i], d0);
#pragma unroll
            for (int o = LPR / 2; o > 0; o >>= 1) d0 += __shfl_xor_sync(0xffffffffu, d0, o);
            const bool ok = r0 + u * RPI + grp < r_end;
            s[u] = ok ? d0 : -INFINITY;
            smax = fmaxf(smax, s[u]);
        }
        const float m_new = fmaxf(m, smax);
        if (m_new > -INFINITY) {
            const float resc = exp2f(m - m_new);             // m = -inf gives 0
            z *= resc;
#pragma unroll
            for (int i = 0; i < 8; ++i) acc[i] *= resc;
#pragma unroll
            for (int u = 0; u < kUnroll; ++u) {
                const float e = exp2f(s[u] - m_new);         // masked rows: exp2(-inf) = 0
                z += e;
                float x[8];
                unpack8(vv[u], x);
#pragma unroll
                for (int i = 0; i < 8; ++i) acc[i] = fmaf(e, x[i], acc[i]);
            }
            m = m_new;
        }
    }

    // merge the lane groups of a warp (lanes that hold the same column slice)
#pragma unroll
    for (int o = 16; o >= LPR; o >>= 1) {
        const float m_o = __shfl_xor_sync(0xffffffffu, m, o);
        const float z_o = __shfl_xor_sync(0xffffffffu, z, o);
        const float m_n = fmaxf(m, m_o);
        const float a = m_n > -INFINITY ? exp2f(m - m_n) : 0.f;
        const float c = m_n > -INFINITY ? exp2f(m_o - m_n) : 0.f;
        z = z * a + z_o * c;
#pragma unroll
        for (int i = 0; i < 8; ++i) {
            const float acc_o = __shfl_xor_sync(0xffffffffu, acc[i], o);
            acc[i] = acc[i] * a + acc_o * c;
        }
        m = m_n;
    }
    // merge the warps of the CTA
    __shared__ float sm_m[kWarps], sm_z[kWarps], sm_acc[kWarps][DH];
    if (grp == 0) {
#pragma unroll
        for (int i = 0; i < 8; ++i) sm_acc[warp][sub * 8 + i] = acc[i];
        if (sub == 0) { sm_m[warp] = m; sm_z[warp] = z; }
    }
    __syncthreads();
    if (threadIdx.x < DH) {
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) M = fmaxf(M, sm_m[w]);
        float Z = 0.f, A = 0.f;
#pragma unroll
        for (int w = 0; w < kWarps; ++w) {
            const float f = M > -INFINITY ? exp2f(sm_m[w] - M) : 0.f;
            Z = fmaf(sm_z[w], f, Z);
            A = fmaf(sm_acc[w][threadIdx.x], f, A);
        }
        float* out = p.partial + (long long)blockIdx.x * (DH + 2);
        out[2 + threadIdx.x] = A;
        if (threadIdx.x == 0) { out[0] = M; out[1] = Z; }
    }
}

template <int DH>
__global__ void __launch_bounds__(DH) decode_combine_kernel(const DecodeParams p) {
    const long long bh = blockIdx.x;
    const int b = (int)(bh / p.H);
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const float* part = p.partial + bh * p.total_chunks * (DH + 2);
    float lam[3];
#pragma unroll
    for (int l = 0; l < 3; ++l) lam[l] = p.gate[b * 3 + l];
    const long long c1 = p.n_chunks[0], c2 = c1 + p.n_chunks[1];
    // global maximum over the chunks that count (gate > 0 and something summed): warp shuffles, then
    // one shared-memory hop across the CTA's warps
    float M = -INFINITY;
    for (long long c = tid; c < p.total_chunks; c += DH) {
        const float g = c < c1 ? lam[0] : (c < c2 ? lam[1] : lam[2]);
        const float mc = part[c * (DH + 2)], zc = part[c * (DH + 2) + 1];
        if (g > 0.f && zc > 0.f) M = fmaxf(M, mc);
    }
    M = warp_max(M);
    __shared__ float sm[DH / 32];
    if (lane == 0) sm[warp] = M;
    __syncthreads();
    M = sm[0];
#pragma unroll
    for (int w = 1; w < DH / 32; ++w) M = fmaxf(M, sm[w]);

    // Weights of a batch of DH chunks are worked out side by side (one chunk per thread) and parked in shared
    // memory; the accumulation over the batch then runs without a branch, its loads independent of each other.
    float Z = 0.f, A = 0.f;
    __shared__ float sw[DH];
    if (M > -INFINITY) {
        for (long long c0 = 0; c0 < p.total_chunks; c0 += DH) {
            const long long c = c0 + tid;
            float w = 0.f;
            if (c < p.total_chunks) {
                const float g = c < c1 ? lam[0] : (c < c2 ? lam[1] : lam[2]);
                const float mc = part[c * (DH + 2)], zc = part[c * (DH + 2) + 1];
                if (g > 0.f && zc > 0.f) { w = g * exp2f(mc - M); Z = fmaf(w, zc, Z); }
            }
            __syncthreads();                                   // the previous batch has been consumed
            sw[tid] = w;
            __syncthreads();
            const int nb = p.total_chunks - c0 < DH ? (int)(p.total_chunks - c0) : DH;
            const float* col = part + c0 * (DH + 2) + 2 + tid;
            int j = 0;
            for (; j + 8 <= nb; j += 8) {
                float v[8];
#pragma unroll
                for (int u = 0; u < 8; ++u) v[u] = col[(long long)(j + u) * (DH + 2)];
#pragma unroll
                for (int u = 0; u < 8; ++u) A = fmaf(sw[j + u], v[u], A);
            }
            for (; j < nb; ++j) A = fmaf(sw[j], col[(long long)j * (DH + 2)], A);
        }
    }
    // Z: every thread holds the share of its own chunks
    Z = warp_sum(Z);
    __shared__ float sz[DH / 32];
    if (lane == 0) sz[warp] = Z;
    __syncthreads();
    Z = 0.f;
#pragma unroll
    for (int w = 0; w < DH / 32; ++w) Z += sz[w];
    __nv_bfloat16* O = static_cast<__nv_bfloat16*>(p.O) + bh * DH;
    O[tid] = __float2bfloat16_rn(Z > 0.f ? A / Z : 0.f);
    if (p.LSE && tid == 0) p.LSE[bh] = Z > 0.f ? (M + log2f(Z)) * kLn2 : -INFINITY;
}

template <int DH>
cudaError_t launch_t(const DecodeParams& p, cudaStream_t st) {
    const long long bh = (long long)p.B * p.H;
    if (bh == 0) return cudaSuccess;
    if (p.total_chunks > 0) {
        decode_partial_kernel<DH><<<(unsigned)(bh * p.total_chunks), kWarps * 32, 0, st>>>(p);
        cudaError_t e = cudaGetLastError();
        if (e != cudaSuccess) return e;
    }
    decode_combine_kernel<DH><<<(unsigned)bh, DH, 0, st>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_decode_combine(const DecodeParams& p, cudaStream_t st) {
    const long long bh = (long long)p.B * p.H;
    if (bh == 0) return cudaSuccess;
    if (p.d == 128) decode_combine_kernel<128><<<(unsigned)bh, 128, 0, st>>>(p);
    else if (p.d == 64) decode_combine_kernel<64><<<(unsigned)bh, 64, 0, st>>>(p);
    else return cudaErrorNotSupported;
    return cudaGetLastError();
}

cudaError_t launch_decode(const DecodeParams& p, cudaStream_t st) {
    if (p.d == 128) return launch_t<128>(p, st);
    if (p.d == 64) return launch_t<64>(p, st);
    return cudaErrorNotSupported;
}

}  // namespace mka

// ---------------------------------------------------------------------------------------------
// mka_decode_static: the decode entry point for callers that cannot hand over scratch memory.
// The per-chunk partials live in the file-scope device array below instead of a caller workspace.
// Every GPU that loads this library carries the array (8 MiB) until the process exits.
namespace mka {
namespace {

constexpr size_t kStaticScratchFloats = (size_t)2 << 20;                    // 2 Mi floats = 8 MiB
static __device__ __align__(256) float g_decode_static_scratch[kStaticScratchFloats];

constexpr int kMaxDevices = 64;
float* g_static_scratch_ptr[kMaxDevices];       // device address of the array, per device ordinal
std::mutex g_static_scratch_mutex;

// In host code the array's name is only a handle; the address a kernel can use has to be asked for,
// once per device and with that device current.  With CUDA's lazy module loading that request (or the first
// launch from this file) is also the moment the 8 MiB are really taken on that device, so it can fail when the
// device has no memory left: the caller then sees MKA_ERR_CUDA from its first call.  The remembered address
// belongs to the device's current context and is not refreshed after a cudaDeviceReset.
cudaError_t static_scratch_address(float** out) {
    int dev = -1;
    cudaError_t e = cudaGetDevice(&dev);
    if (e != cudaSuccess) return e;
    if (dev < 0 || dev >= kMaxDevices) return cudaErrorInvalidDevice;
    std::lock_guard<std::mutex> lock(g_static_scratch_mutex);
    if (!g_static_scratch_ptr[dev]) {
        float* ptr = nullptr;
        e = cudaGetSymbolAddress(reinterpret_cast<void**>(&ptr), g_decode_static_scratch);
        if (e != cudaSuccess) return e;
        if (!ptr) return cudaErrorInvalidSymbol;
        g_static_scratch_ptr[dev] = ptr;
    }
    *out = g_static_scratch_ptr[dev];
    return cudaSuccess;
}

inline bool is_aligned16(const void* p) { return (reinterpret_cast<uintptr_t>(p) & 15u) == 0; }

}  // namespace
}  // namespace mka

extern "C" size_t mka_decode_static_max_bytes(void) { return mka::kStaticScratchFloats * sizeof(float); }

extern "C" mka_status mka_decode_static(const mka_shape* s, const void* q, const mka_level L[3], const float* gate,
                                        void* O, float* LSE, void* stream) {
    using namespace mka;
    if (!s || !L) return MKA_ERR_ARG;
    if (s->dtype != MKA_BF16 || s->mode != MKA_MODE_FAST) return MKA_ERR_UNSUPPORTED;
    if (s->B < 0 || s->H < 0 || s->T != 1) return MKA_ERR_SHAPE;
    if (s->d != 64 && s->d != 128) return MKA_ERR_SHAPE;
    if (s->kv_heads < 0 || (s->kv_heads > 0 && (s->H % s->kv_heads != 0))) return MKA_ERR_SHAPE;
    int64_t n_level[3];
    for (int l = 0; l < 3; ++l) {
        n_level[l] = L[l].n;
        if (L[l].n < 0) return MKA_ERR_SHAPE;
        if (L[l].n == 0) continue;
        if (!L[l].k || !L[l].v) return MKA_ERR_ARG;
        if (L[l].stride_n < s->d || L[l].stride_b < 0 || L[l].stride_h < 0) return MKA_ERR_SHAPE;
        if (!is_aligned16(L[l].k) || !is_aligned16(L[l].v)) return MKA_ERR_ALIGN;
        if (L[l].stride_n % 8 || L[l].stride_b % 8 || L[l].stride_h % 8) return MKA_ERR_ALIGN;
    }
    if (s->B == 0 || s->H == 0) return MKA_OK;
    if (!q || !gate || !O) return MKA_ERR_ARG;
    if (!is_aligned16(q) || !is_aligned16(O)) return MKA_ERR_ALIGN;
    mka_decode_plan_t plan;
    mka_status st = mka_decode_plan(n_level, s->B, s->H, s->d, &plan);
    if (st != MKA_OK) return st;
    const unsigned long long slots = (unsigned long long)s->B * s->H * (unsigned long long)plan.total_chunks;
    if (slots > 0x7fffffffULL) return MKA_ERR_SHAPE;
    // the split table of this problem needs more partial slots than the built-in array holds
    if (slots * (unsigned long long)(s->d + 2) > kStaticScratchFloats) return MKA_ERR_WORKSPACE;
    float* scratch = nullptr;
    if (static_scratch_address(&scratch) != cudaSuccess) return MKA_ERR_CUDA;
    DecodeParams p;
    p.q = q; p.O = O; p.LSE = LSE; p.gate = gate;
    for (int l = 0; l < 3; ++l) {
        p.L[l].k = L[l].k; p.L[l].v = L[l].v; p.L[l].n = L[l].n;
        p.L[l].sb = L[l].stride_b; p.L[l].sh = L[l].stride_h; p.L[l].sn = L[l].stride_n;
        p.n_chunks[l] = plan.n_chunks[l];
    }
    p.B = s->B; p.H = s->H; p.d = s->d;
    p.kv_group = s->kv_heads > 0 ? s->H / s->kv_heads : 1;
    p.scale = s->scale > 0.f ? s->scale : 1.0f / sqrtf((float)s->d);
    p.chunk_rows = plan.chunk_rows;
    p.total_chunks = plan.total_chunks;
    // Nothing in the array has to start at zero: the partial kernel writes every slot that the combine
    // kernel of the same call reads, so whatever an earlier call left behind is never looked at.
    p.partial = scratch;
    cudaError_t e = launch_decode(p, static_cast<cudaStream_t>(stream));
    if (e == cudaErrorNotSupported) return MKA_ERR_UNSUPPORTED;
    return e == cudaSuccess ? MKA_OK : MKA_ERR_CUDA;
}
