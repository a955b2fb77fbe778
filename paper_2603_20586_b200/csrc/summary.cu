// Causal L2 session summary (Alg. 1, the loop that fills M_2; Alg. 2 step 3): row t of the output summarises
// X[:, :t+1] as a prefix mean or as an exponential moving average.  A scan along the sequence, HBM-bound: X is read
// once and M2 written once.
//
// One CTA owns a strip of kNC columns of one batch element for the WHOLE sequence and walks it in 32 KB tiles (256 or 512 rows):
// no CTA ever waits for another.  The tiles arrive through a ring of TMA loads (the strip's rows are 32..128
// contiguous bytes, a row apart in memory), so every CTA keeps three 16 KB tiles of reads in flight and three CTAs share an SM.  Inside a tile the 256
// threads are kNC columns x G row groups: each thread scans its rows/G rows of one column in registers, the groups'
// totals are combined through shared memory (both summaries are affine recurrences state' = a state + b, so a
// group's effect is the pair (a^rows, b)), the results go back to shared memory and leave as 16-byte row-contiguous
// stores.  The running state of each column is carried from tile to tile in shared memory and can be carried from
// call to call through `state` (a session processed in chunks).
#include "tc_ptx.cuh"

namespace mka {
namespace {

constexpr int kSumThreads = 256;
constexpr int kSumTileBytes = 32768;  // every tile is 16 KB: 512 rows of a 32-byte strip ... 128 rows of a 128-byte strip
constexpr int kSumMaxStages = 5;     // tiles in flight per CTA: 3 (three CTAs per SM) ... 11 (one CTA per SM, 176 KB of reads in flight)

struct SummaryParams {
    void* M2;
    float* state;          // [B, D] in/out, may be null
    long long T, n_prev;
    int B, D, kind;
    float beta;
    int use_state;         // state holds a carried value on entry
    int stages;            // depth of the tile ring
    unsigned int* status;  // may be null
    unsigned long long wait_limit_ns;
};

// two adjacent columns of a row at once
template <typename T> struct Pair;
template <> struct Pair<__nv_bfloat16> {
    using type = uint32_t;
    static __device__ __forceinline__ void unpack(uint32_t w, float& lo, float& hi) {
        lo = __uint_as_float(w << 16); hi = __uint_as_float(w & 0xffff0000u);
    }
    static __device__ __forceinline__ uint32_t pack(float lo, float hi) {
        const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
        return *reinterpret_cast<const uint32_t*>(&v);
    }
};
template <> struct Pair<float> {
    using type = float2;
    static __device__ __forceinline__ void unpack(float2 w, float& lo, float& hi) { lo = w.x; hi = w.y; }
    static __device__ __forceinline__ float2 pack(float lo, float hi) { return make_float2(lo, hi); }
};

template <typename T, int kNC, bool kEma>
__global__ void __launch_bounds__(kSumThreads, 3) l2_summary_kernel(const __grid_constant__ CUtensorMap map, const SummaryParams p) {
    using P2 = typename Pair<T>::type;
    constexpr int kRows = kSumTileBytes / (kNC * (int)sizeof(T));   // rows per tile: large, to amortise the per-tile barriers
    constexpr int kNP = kNC / 2;                      // column pairs of the strip
    constexpr int G = kSumThreads / kNP;              // row groups
    constexpr int RG = kRows / G;                     // rows of a tile scanned by one thread
    static_assert(RG >= 1 && RG * G == kRows, "tile geometry");
    constexpr uint32_t kTileBytes = kSumTileBytes;
    constexpr int kVecPerRow = kNC * sizeof(T) / 16;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 127) & ~static_cast<uintptr_t>(127));
    const int kSumStages = p.stages;
    uint8_t* ring = smem;                                                   // p.stages tiles [kRows][kNC]
    P2* otile = reinterpret_cast<P2*>(smem + kSumStages * kTileBytes);      // [kRows][kNP]
    __shared__ float2 part[G][kNP];
    __shared__ float2 carry[kNP];
    __shared__ uint64_t full[kSumMaxStages];
    __shared__ WaitCtl wait_ctl;

    const int tid = threadIdx.x;
    const int c = tid % kNP, g = tid / kNP;           // column pair, row group
    const int col0 = blockIdx.x * kNC;
    const int b = blockIdx.y;
    const int ntiles = (int)((p.T + kRows - 1) / kRows);
    const int Tn = (int)p.T;                          // the entry point keeps T below 2^31
    const float beta = p.beta, omb = 1.f - p.beta;

    if (tid == 0) {
        wait_ctl.abort = 0;
        wait_ctl.limit_ns = p.wait_limit_ns;
        for (int s = 0; s < kSumMaxStages; ++s) mbar_init(&full[s], 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (tid < kNP) {
        float2 v = make_float2(0.f, 0.f);
        if (p.use_state) {
            const float* st = p.state + (long long)b * p.D + col0 + 2 * tid;
            if (col0 + 2 * tid < p.D) v.x = st[0];
            if (col0 + 2 * tid + 1 < p.D) v.y = st[1];
        }
        carry[tid] = v;
    }
    __syncthreads();
    volatile WaitCtl* abortp = &wait_ctl;
    // a box of the tensor map holds at most 256 rows: taller tiles arrive as consecutive boxes on the same barrier
    constexpr int kBoxRows = kRows > 256 ? 256 : kRows;
    auto load_tile = [&](uint8_t* dst, int row0, uint64_t* bar) {
#pragma unroll
        for (int r = 0; r < kRows; r += kBoxRows)
            tma_load_3d(dst + (size_t)r * kNC * sizeof(T), &map, col0, row0 + r, b, bar);
    };
    if (tid == 0) {
        for (int i = 0; i < kSumStages && i < ntiles; ++i) {
            mbar_expect_tx(&full[i], kTileBytes);
            load_tile(ring + i * kTileBytes, i * kRows, &full[i]);
        }
    }
    // Both summaries are affine in the state: state' = a state + b.  a of a full group of RG rows:
    float a_rg = 1.f;
    if (kEma) {
#pragma unroll
        for (int k = 0; k < RG; ++k) a_rg *= beta;
    }
    const bool fresh_ema = kEma && !p.use_state;      // the first token of the session initialises the average
    bool ok = true;
    int s = 0;
    uint32_t phase = 0;                               // ring slot of tile i and the parity of its use
    for (int i = 0; i < ntiles; ++i) {
        ok = mbar_wait(&full[s], phase, abortp);
        if (!__syncthreads_and(ok)) { ok = false; break; }
        const P2* tile = reinterpret_cast<const P2*>(ring + (size_t)s * kTileBytes) + (size_t)g * RG * kNP + c;
        const int t0 = i * kRows + g * RG;                               // first row of this thread's group
        const int left = Tn - t0;
        const int nv = left >= RG ? RG : (left > 0 ? left : 0);          // valid rows of the group (RG except in the last tile)
        if (i == 0 && fresh_ema && g == 0) {                             // m_{-1} := x_0 makes m_0 = x_0
            float2 v;
            Pair<T>::unpack(tile[0], v.x, v.y);
            carry[c] = v;
        }
        // scan of this thread's rows of its two columns, with a zero incoming state
        float l0[RG], l1[RG];
        float r0 = 0.f, r1 = 0.f;
#pragma unroll
        for (int k = 0; k < RG; ++k) {
            float x0, x1;
            Pair<T>::unpack(tile[k * kNP], x0, x1);
            if (nv == RG || k < nv) {
                if (kEma) { r0 = fmaf(beta, r0, omb * x0); r1 = fmaf(beta, r1, omb * x1); }
                else { r0 += x0; r1 += x1; }
            }
            l0[k] = r0; l1[k] = r1;
        }
        part[g][c] = make_float2(r0, r1);
        __syncthreads();                                                 // totals (and the fresh carry) visible
        // state entering this group: the carried state pushed through the groups before it
        float2 m = carry[c];
        const bool last_tile = (i + 1) * kRows > Tn;
#pragma unroll
        for (int gg = 0; gg < G; ++gg) {
            if (gg < g) {
                float a = a_rg;
                if (kEma && last_tile) {
                    const int l2 = Tn - (i * kRows + gg * RG);
                    a = l2 >= RG ? a_rg : (l2 > 0 ? powf(beta, (float)l2) : 1.f);
                }
                const float2 pt = part[gg][c];
                m.x = kEma ? fmaf(a, m.x, pt.x) : m.x + pt.x;
                m.y = kEma ? fmaf(a, m.y, pt.y) : m.y + pt.y;
            }
        }
        P2* orow = otile + (size_t)g * RG * kNP + c;
        float apow = beta;
        float cnt = (float)(p.n_prev + (long long)t0 + 1);                          // tokens summarised by row k = 0 (exact below 2^24)
#pragma unroll
        for (int k = 0; k < RG; ++k) {
            float v0, v1;
            if (kEma) { v0 = fmaf(apow, m.x, l0[k]); v1 = fmaf(apow, m.y, l1[k]); apow *= beta; }
            else { const float inv = __fdividef(1.f, cnt); v0 = (m.x + l0[k]) * inv; v1 = (m.y + l1[k]) * inv; cnt += 1.f; }
            orow[k * kNP] = Pair<T>::pack(v0, v1);
        }
        float2 new_carry = make_float2(0.f, 0.f);
        if (g == G - 1) {
            const float a = !kEma ? 1.f : (nv == RG ? a_rg : powf(beta, (float)nv));
            new_carry = make_float2(fmaf(a, m.x, r0), fmaf(a, m.y, r1));
        }
        __syncthreads();                                                 // output tile complete; everybody has read carry
        if (g == G - 1) carry[c] = new_carry;
        // row-contiguous 16-byte stores of the valid rows
        T* out = static_cast<T*>(p.M2) + ((long long)b * p.T + (long long)i * kRows) * p.D + col0;
#pragma unroll
        for (int v = tid; v < kRows * kVecPerRow; v += kSumThreads) {
            const int r = v / kVecPerRow, q = v % kVecPerRow;
            if (i * kRows + r < Tn && col0 + q * (int)(16 / sizeof(T)) < p.D)
                *reinterpret_cast<uint4*>(reinterpret_cast<uint8_t*>(out + (long long)r * p.D) + q * 16) =
                    *reinterpret_cast<const uint4*>(reinterpret_cast<const uint8_t*>(otile) + (size_t)v * 16);
        }
        __syncthreads();                                                 // ring slot and output tile free again
        if (tid == 0 && i + kSumStages < ntiles) {
            mbar_expect_tx(&full[s], kTileBytes);
            load_tile(ring + s * kTileBytes, (i + kSumStages) * kRows, &full[s]);
        }
        if (++s == kSumStages) { s = 0; phase ^= 1u; }
    }
    if (!ok && tid == 0) {
        // copies issued but not consumed must land before the shared memory is given up (bounded)
        for (int s = 0; s < kSumStages; ++s) mbar_wait(&full[s], 0, abortp), mbar_wait(&full[s], 1, abortp);
        if (p.status) atomicExch(p.status, (unsigned int)MKA_ERR_TIMEOUT);
    }
    __syncthreads();
    if (ok && p.state && tid < kNP) {
        float* st = p.state + (long long)b * p.D + col0 + 2 * tid;
        if (col0 + 2 * tid < p.D) st[0] = carry[tid].x;
        if (col0 + 2 * tid + 1 < p.D) st[1] = carry[tid].y;
    }
}

template <typename T, int kNC, bool kEma>
cudaError_t launch_k(const CUtensorMap& map, const SummaryParams& p, size_t smem, cudaStream_t st) {
    cudaError_t e = cudaFuncSetAttribute(l2_summary_kernel<T, kNC, kEma>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    dim3 grid((p.D + kNC - 1) / kNC, p.B);
    l2_summary_kernel<T, kNC, kEma><<<grid, kSumThreads, smem, st>>>(map, p);
    return cudaGetLastError();
}

template <typename T, int kNC>
cudaError_t launch_t(const void* X, const SummaryParams& p, cudaStream_t st) {
    CUtensorMap map;
    constexpr int kRows = kSumTileBytes / (kNC * (int)sizeof(T));
    static_assert(kRows <= 1024, "tile geometry");
    if (!make_strip_map(&map, X, sizeof(T) == 2, p.D, p.T, p.B, kNC, kRows > 256 ? 256 : kRows)) return cudaErrorNotSupported;
    const size_t smem = (size_t)(p.stages + 1) * kSumTileBytes + 128;
    return p.kind == MKA_SUMMARY_EMA ? launch_k<T, kNC, true>(map, p, smem, st) : launch_k<T, kNC, false>(map, p, smem, st);
}

}  // namespace

cudaError_t launch_l2_summary(const void* X, void* M2, float* state, int use_state, long long n_prev, int B, long long T, int D,
                              int dtype, int kind, float beta, unsigned int* status, cudaStream_t st) {
    if (B == 0 || T == 0 || D == 0) return cudaSuccess;
    if (!tensor_map_encoder_available()) return cudaErrorNotSupported;
    SummaryParams p;
    p.M2 = M2; p.state = state; p.T = T; p.n_prev = n_prev; p.B = B; p.D = D; p.kind = kind; p.beta = beta;
    p.use_state = use_state; p.status = status; p.wait_limit_ns = wait_limit_ns();
    // Strips as wide as possible (whole 128-byte lines per row are kindest to DRAM) while most SMs still get a CTA;
    // the fewer CTAs share an SM, the deeper each one's ring of tiles in flight.
    const long long want = 120;
    auto ctas = [&](int nc) { return (long long)B * ((D + nc - 1) / nc); };
    auto depth = [&](int nc) {
        const long long per_sm = (ctas(nc) + 147) / 148;
        long long st_ = (200 * 1024 / (per_sm > 3 ? 3 : per_sm) - kSumTileBytes) / kSumTileBytes;
        return (int)(st_ > kSumMaxStages ? kSumMaxStages : (st_ < 2 ? 2 : st_));
    };
    if (dtype == MKA_F32) {
        if (ctas(32) >= want) { p.stages = depth(32); return launch_t<float, 32>(X, p, st); }
        if (ctas(16) >= want) { p.stages = depth(16); return launch_t<float, 16>(X, p, st); }
        { p.stages = depth(8); return launch_t<float, 8>(X, p, st); }
    }
    if (ctas(64) >= want) { p.stages = depth(64); return launch_t<__nv_bfloat16, 64>(X, p, st); }
    if (ctas(32) >= want) { p.stages = depth(32); return launch_t<__nv_bfloat16, 32>(X, p, st); }
    { p.stages = depth(16); return launch_t<__nv_bfloat16, 16>(X, p, st); }
}

}  // namespace mka
