// Causal L2 session summary (Alg. 1, the loop that fills M_2; Alg. 2 step 3): row t of the output summarises
// X[:, :t+1] as a prefix mean or as an exponential moving average.  A scan along the sequence, HBM-bound: X is read
// once and M2 written once.
//
// One CTA owns a strip of kNC columns of one batch element for the WHOLE sequence and walks it in tiles of 128 rows:
// no CTA ever waits for another.  The tiles arrive through a ring of TMA loads (the strip's rows are 64..128
// contiguous bytes, a row apart in memory), so a CTA keeps ~100 KB of reads in flight.  Inside a tile the 512
// threads are kNC columns x G row groups: each thread scans its 128/G rows of one column in registers, the groups'
// totals are combined through shared memory (both summaries are affine recurrences state' = a state + b, so a
// group's effect is the pair (a^rows, b)), the results go back to shared memory and leave as 16-byte row-contiguous
// stores.  The running state of each column is carried from tile to tile in shared memory and can be carried from
// call to call through `state` (a session processed in chunks).
#include "tc_ptx.cuh"

namespace mka {
namespace {

constexpr int kSumThreads = 512;
constexpr int kRows = 128;            // rows per tile
constexpr int kSumStages = 6;

struct SummaryParams {
    void* M2;
    float* state;          // [B, D] in/out, may be null
    long long T, n_prev;
    int B, D, kind;
    float beta;
    int use_state;         // state holds a carried value on entry
    unsigned int* status;  // may be null
};

template <typename T> __device__ __forceinline__ float to_f32(T v);
template <> __device__ __forceinline__ float to_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ float to_f32<__nv_bfloat16>(__nv_bfloat16 v) { return __bfloat162float(v); }
template <typename T> __device__ __forceinline__ T from_f32(float v);
template <> __device__ __forceinline__ float from_f32<float>(float v) { return v; }
template <> __device__ __forceinline__ __nv_bfloat16 from_f32<__nv_bfloat16>(float v) { return __float2bfloat16_rn(v); }

template <typename T, int kNC>
__global__ void __launch_bounds__(kSumThreads, 1) l2_summary_kernel(const __grid_constant__ CUtensorMap map, const SummaryParams p) {
    constexpr int G = kSumThreads / kNC;              // row groups
    constexpr int RG = kRows / G;                     // rows of a tile scanned by one thread
    constexpr uint32_t kTileBytes = kRows * kNC * sizeof(T);
    constexpr int kVecPerRow = kNC * sizeof(T) / 16;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~static_cast<uintptr_t>(127));
    T* ring = reinterpret_cast<T*>(smem);                                   // kSumStages tiles [kRows][kNC]
    T* otile = reinterpret_cast<T*>(smem + kSumStages * kTileBytes);        // [kRows][kNC]
    __shared__ float part[G][kNC];
    __shared__ float carry[kNC];
    __shared__ uint64_t full[kSumStages];
    __shared__ int abort_flag;

    const int tid = threadIdx.x;
    const int c = tid % kNC, g = tid / kNC;
    const int col0 = blockIdx.x * kNC;
    const int b = blockIdx.y;
    const long long ntiles = (p.T + kRows - 1) / kRows;
    const bool ema = p.kind == MKA_SUMMARY_EMA;
    const float beta = p.beta, omb = 1.f - p.beta;

    if (tid == 0) {
        abort_flag = 0;
        for (int s = 0; s < kSumStages; ++s) mbar_init(&full[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < kNC) carry[tid] = (p.use_state && col0 + tid < p.D) ? p.state[(long long)b * p.D + col0 + tid] : 0.f;
    __syncthreads();
    volatile int* abortp = &abort_flag;
    if (tid == 0) {
        for (int i = 0; i < kSumStages && i < ntiles; ++i) {
            mbar_expect_tx(&full[i], kTileBytes);
            tma_load_3d(reinterpret_cast<uint8_t*>(ring) + i * kTileBytes, &map, col0, i * kRows, b, &full[i]);
        }
    }
    // a^RG of a full group (EMA); partial groups of the last tile use their own power
    float beta_rg = 1.f;
    if (ema) {
#pragma unroll
        for (int k = 0; k < RG; ++k) beta_rg *= beta;
    }
    const bool fresh_ema = ema && !p.use_state;       // the first token of the session initialises the average
    bool ok = true;
    for (long long i = 0; i < ntiles; ++i) {
        const int s = (int)(i % kSumStages);
        ok = mbar_wait(&full[s], (uint32_t)(i / kSumStages) & 1u, abortp);
        if (!__syncthreads_and(ok)) { ok = false; break; }
        const T* tile = ring + (size_t)s * kRows * kNC;
        const long long t0 = i * kRows + (long long)g * RG;              // first row of this thread's group
        long long left = p.T - t0;
        const int nv = left >= RG ? RG : (left > 0 ? (int)left : 0);     // valid rows of the group
        if (i == 0 && fresh_ema && g == 0) carry[c] = to_f32<T>(tile[c]);   // m_{-1} := x_0 makes m_0 = x_0
        // scan of this thread's rows with a zero incoming state
        float loc[RG];
        float run = 0.f;
#pragma unroll
        for (int k = 0; k < RG; ++k) {
            const float x = to_f32<T>(tile[(g * RG + k) * kNC + c]);
            if (k < nv) run = ema ? fmaf(beta, run, omb * x) : run + x;
            loc[k] = run;
        }
        part[g][c] = run;
        __syncthreads();                                                 // totals (and the fresh carry) visible
        // state entering this group: the carried state pushed through the groups before it
        float m_in = carry[c];
#pragma unroll
        for (int gg = 0; gg < G; ++gg) {
            if (gg < g) {
                long long l2 = p.T - (i * kRows + (long long)gg * RG);
                const float a = !ema ? 1.f : (l2 >= RG ? beta_rg : (l2 > 0 ? powf(beta, (float)l2) : 1.f));
                m_in = fmaf(a, m_in, part[gg][c]);
            }
        }
        float apow = beta;
#pragma unroll
        for (int k = 0; k < RG; ++k) {
            float v;
            if (ema) { v = fmaf(apow, m_in, loc[k]); apow *= beta; }
            else v = (m_in + loc[k]) / (float)(p.n_prev + t0 + k + 1);
            otile[(g * RG + k) * kNC + c] = from_f32<T>(v);
        }
        float new_carry = 0.f;
        if (g == G - 1) {
            const float a = !ema ? 1.f : (nv == RG ? beta_rg : powf(beta, (float)nv));
            new_carry = fmaf(a, m_in, run);
        }
        __syncthreads();                                                 // output tile complete; everybody has read carry
        if (g == G - 1) carry[c] = new_carry;
        // row-contiguous 16-byte stores of the valid rows
        T* out = static_cast<T*>(p.M2) + ((long long)b * p.T + i * kRows) * p.D + col0;
        for (int v = tid; v < kRows * kVecPerRow; v += kSumThreads) {
            const int r = v / kVecPerRow, q = v % kVecPerRow;
            if (i * kRows + r < p.T && col0 + q * (int)(16 / sizeof(T)) < p.D)
                *reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(out + (long long)r * p.D) + q * 16) =
                    *reinterpret_cast<const uint4*>(reinterpret_cast<const uint8_t*>(otile) + (size_t)(r * kVecPerRow + q) * 16);
        }
        __syncthreads();                                                 // ring slot and output tile free again
        if (tid == 0 && i + kSumStages < ntiles) {
            mbar_expect_tx(&full[s], kTileBytes);
            tma_load_3d(reinterpret_cast<uint8_t*>(ring) + s * kTileBytes, &map, col0, (int)((i + kSumStages) * kRows), b, &full[s]);
        }
    }
    if (!ok && tid == 0) {
        // copies issued but not consumed must land before the shared memory is given up (bounded)
        for (int s = 0; s < kSumStages; ++s) mbar_wait(&full[s], 0, abortp), mbar_wait(&full[s], 1, abortp);
        if (p.status) atomicExch(p.status, (unsigned int)MKA_ERR_TIMEOUT);
    }
    __syncthreads();
    if (ok && p.state && tid < kNC && col0 + tid < p.D) p.state[(long long)b * p.D + col0 + tid] = carry[tid];
}

template <typename T, int kNC>
cudaError_t launch_t(const void* X, const SummaryParams& p, cudaStream_t st) {
    CUtensorMap map;
    if (!make_strip_map(&map, X, sizeof(T) == 2, p.D, p.T, p.B, kNC, kRows)) return cudaErrorNotSupported;
    const size_t smem = (size_t)(kSumStages + 1) * kRows * kNC * sizeof(T) + 128;
    cudaError_t e = cudaFuncSetAttribute(l2_summary_kernel<T, kNC>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    dim3 grid((p.D + kNC - 1) / kNC, p.B);
    l2_summary_kernel<T, kNC><<<grid, kSumThreads, smem, st>>>(map, p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_l2_summary(const void* X, void* M2, float* state, int use_state, long long n_prev, int B, long long T, int D,
                              int dtype, int kind, float beta, unsigned int* status, cudaStream_t st) {
    if (B == 0 || T == 0 || D == 0) return cudaSuccess;
    if (!tensor_map_encoder_available()) return cudaErrorNotSupported;
    SummaryParams p;
    p.M2 = M2; p.state = state; p.T = T; p.n_prev = n_prev; p.B = B; p.D = D; p.kind = kind; p.beta = beta;
    p.use_state = use_state; p.status = status;
    if (dtype == MKA_F32) return launch_t<float, 32>(X, p, st);
    // bf16: 128-byte strips when that still gives every SM a CTA, 64-byte strips otherwise
    if ((long long)B * ((D + 63) / 64) >= 148 && D % 64 == 0) return launch_t<__nv_bfloat16, 64>(X, p, st);
    return launch_t<__nv_bfloat16, 32>(X, p, st);
}

}  // namespace mka
