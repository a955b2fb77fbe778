// Split-KV single-token decode of Eq. 5 over PAGED levels with grouped-query sharing of the KV heads (the serving
// layout of the paper's inference setup: GQA models, paged KV cache for long contexts).
//
// One CTA = (sequence, KV head, chunk of one level).  All G = H / H_kv query heads that share the KV head ride in the
// 16 rows of one warp-level matrix product, so every cached row is read from HBM once per KV head instead of once
// per query head.  Rows are found through the page table (row r -> page table[r / page_rows], offset r % page_rows)
// (the chunk's slice of the table is read into shared memory once) and brought into shared memory with 16-byte
// asynchronous copies, three 64-row tiles in flight; each of the four
// warps owns 16 rows of a tile:
//     S[16 x 16]  = Q[16 x d] K^T          (mma m16n8k16, bf16 in, fp32 out; K through ldmatrix)
//     p = 2^(c S - m) with the running maximum of Eq. 11-14 per query head, z += sum p
//     O[16 x d]  += P[16 x 16] V[16 x d]   (P straight from the S registers; V through ldmatrix.trans)
// The warps' (m, z, O) are merged through shared memory into one UN-GATED partial per (query head, chunk) in the
// layout of the dense decode, and the same gate-weighted combine kernel finishes the job.
// A level whose gate is exactly 0 for a sequence (hard top-k routing) is not read at all.
#include "common.cuh"

namespace mka {
namespace {

constexpr int kThreads = 128;
constexpr int kTileRows = 64;
constexpr int kStages = 3;
constexpr int kSliceCap = 1024;                      // page-table entries of a chunk kept in shared memory

__device__ __forceinline__ uint32_t smem_addr(const void* p) { return (uint32_t)__cvta_generic_to_shared(p); }
__device__ __forceinline__ void cp_async16(uint32_t dst, const void* src) {
    asm volatile("cp.async.cg.shared.global [%0], [%1], 16;" ::"r"(dst), "l"(src) : "memory");
}
__device__ __forceinline__ void cp_async_commit() { asm volatile("cp.async.commit_group;" ::: "memory"); }
template <int N> __device__ __forceinline__ void cp_async_wait() { asm volatile("cp.async.wait_group %0;" ::"n"(N) : "memory"); }
__device__ __forceinline__ void ldmatrix_x4(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void ldmatrix_x4_trans(uint32_t addr, uint32_t (&r)[4]) {
    asm volatile("ldmatrix.sync.aligned.m8n8.x4.trans.shared.b16 {%0,%1,%2,%3}, [%4];"
                 : "=r"(r[0]), "=r"(r[1]), "=r"(r[2]), "=r"(r[3]) : "r"(addr));
}
__device__ __forceinline__ void mma_bf16(float (&c)[4], const uint32_t (&a)[4], uint32_t b0, uint32_t b1) {
    asm volatile("mma.sync.aligned.m16n8k16.row.col.f32.bf16.bf16.f32 {%0,%1,%2,%3}, {%4,%5,%6,%7}, {%8,%9}, {%0,%1,%2,%3};"
                 : "+f"(c[0]), "+f"(c[1]), "+f"(c[2]), "+f"(c[3])
                 : "r"(a[0]), "r"(a[1]), "r"(a[2]), "r"(a[3]), "r"(b0), "r"(b1));
}
__device__ __forceinline__ uint32_t pack2(float lo, float hi) {
    const __nv_bfloat162 v = __floats2bfloat162_rn(lo, hi);
    return *reinterpret_cast<const uint32_t*>(&v);
}

template <int DH>
__global__ void __launch_bounds__(kThreads, 2) decode_paged_kernel(const DecodePagedParams p) {
    constexpr int kPitch = DH * 2 + 16;                     // bytes between rows in shared memory: ldmatrix hits every bank once
    constexpr int kTileBytes = kTileRows * kPitch;          // one of K or V
    constexpr int kVecPerRow = DH / 8;                      // 16-byte pieces of a row
    constexpr int kRowsPerPass = kThreads / kVecPerRow;
    constexpr int KS = DH / 16;                             // k-steps of Q K^T
    constexpr int NB = DH / 8;                              // 8-column blocks of O
    extern __shared__ __align__(128) uint8_t smem[];

    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int g = lane >> 2, t = lane & 3;
    const int G = p.H / p.H_kv;                             // query heads per KV head, <= 16
    long long chunk = blockIdx.x % p.total_chunks;
    const long long bk = blockIdx.x / p.total_chunks;
    const int b = (int)(bk / p.H_kv), kvh = (int)(bk % p.H_kv);
    const long long chunk_all = chunk;
    int lvl = 0;
    while (lvl < 2 && chunk >= p.n_chunks[lvl]) { chunk -= p.n_chunks[lvl]; ++lvl; }
    const PagedLevelDev L = p.L[lvl];
    long long n_b = L.rows ? (long long)L.rows[b] : L.n;                       // valid rows of this sequence
    n_b = n_b < 0 ? 0 : (n_b > L.n ? L.n : n_b);
    const long long r_begin = chunk * p.chunk_rows;
    long long r_end = r_begin + p.chunk_rows < n_b ? r_begin + p.chunk_rows : n_b;
    const bool skip = p.gate[b * 3 + lvl] == 0.f || r_end <= r_begin;
    float* part0 = p.partial + (((long long)b * p.H + (long long)kvh * G) * p.total_chunks + chunk_all) * (DH + 2);
    const long long part_stride = p.total_chunks * (DH + 2);                   // from one query head to the next
    if (skip) {                                                                // nothing to read: empty partials
        for (int r = 0; r < G; ++r) {
            float* out = part0 + r * part_stride;
            for (int i = tid; i < DH + 2; i += kThreads) out[i] = i == 0 ? -INFINITY : 0.f;
        }
        return;
    }

    // Q fragments of the group's heads (rows >= G are zero): a[ks] = {Q[g][16ks+2t..], Q[g+8][..], Q[g][16ks+8+2t..], Q[g+8][..]}
    uint32_t qa[KS][4];
    {
        const __nv_bfloat16* q0 = static_cast<const __nv_bfloat16*>(p.q) + ((long long)b * p.H + (long long)kvh * G) * DH;
#pragma unroll
        for (int ks = 0; ks < KS; ++ks) {
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int row = g + (i & 1) * 8, col = 16 * ks + (i >> 1) * 8 + 2 * t;
                qa[ks][i] = row < G ? *reinterpret_cast<const uint32_t*>(q0 + (long long)row * DH + col) : 0u;
            }
        }
    }
    const float c2 = p.scale * kLog2e;                      // scores in the base-2 domain

    const int shift = L.page_shift;
    const long long page_mask = ((long long)1 << shift) - 1;
    // this chunk's slice of the page table, fetched once: at most one entry per row of the chunk
    __shared__ int s_pages[kSliceCap];
    const long long page0 = r_begin >> shift;
    // (a dense level comes without a table: it is one page per sequence, the page being the batch index)
    const int* table = L.table ? L.table + (long long)b * L.table_stride + (long long)kvh * L.table_head_stride + page0 : nullptr;
    const long long n_pages = ((r_end - 1) >> shift) - page0 + 1;
    const bool sliced = n_pages <= kSliceCap;              // (tiny pages in a long chunk: look the table up in place)
    if (sliced)
        for (int i = tid; i < (int)n_pages; i += kThreads) s_pages[i] = table ? table[i] : b;
    __syncthreads();
    const __nv_bfloat16* Kbase = static_cast<const __nv_bfloat16*>(L.k) + (long long)kvh * L.sh;
    const __nv_bfloat16* Vbase = static_cast<const __nv_bfloat16*>(L.v) + (long long)kvh * L.sh;
    const int piece = tid % kVecPerRow, prow = tid / kVecPerRow;
    auto load_tile = [&](long long tile, int stage) {
        uint8_t* sK = smem + (size_t)stage * 2 * kTileBytes;
        uint8_t* sV = sK + kTileBytes;
        const long long base = r_begin + tile * kTileRows;
#pragma unroll
        for (int pass = 0; pass < kTileRows / kRowsPerPass; ++pass) {
            const int rr = pass * kRowsPerPass + prow;
            long long r = base + rr;
            if (r >= r_end) r = r_end - 1;                  // a tail row re-reads the last valid row (masked later)
            const long long pi = (r >> shift) - page0;
            const long long off = (long long)(sliced ? s_pages[pi] : table[pi]) * L.sp + (r & page_mask) * L.sn + piece * 8;
            cp_async16(smem_addr(sK + rr * kPitch + piece * 16), Kbase + off);
            cp_async16(smem_addr(sV + rr * kPitch + piece * 16), Vbase + off);
        }
    };

    float m[2] = {-INFINITY, -INFINITY}, z[2] = {0.f, 0.f};     // rows g and g + 8
    float o[NB][4];
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) { o[nb][0] = o[nb][1] = o[nb][2] = o[nb][3] = 0.f; }

    const long long n_tiles = (r_end - r_begin + kTileRows - 1) / kTileRows;
#pragma unroll
    for (int s = 0; s < kStages - 1; ++s) {
        if (s < n_tiles) load_tile(s, s);
        cp_async_commit();
    }
    const int kb = warp * 16;                               // this warp's rows of a tile
    for (long long i = 0; i < n_tiles; ++i) {
        cp_async_wait<kStages - 2>();
        __syncthreads();
        if (i + kStages - 1 < n_tiles) load_tile(i + kStages - 1, (int)((i + kStages - 1) % kStages));
        cp_async_commit();
        const uint8_t* sK = smem + (size_t)(i % kStages) * 2 * kTileBytes;
        const uint8_t* sV = sK + kTileBytes;

        float s[2][4];
#pragma unroll
        for (int nb = 0; nb < 2; ++nb) { s[nb][0] = s[nb][1] = s[nb][2] = s[nb][3] = 0.f; }
        {
            // matrices of one ldmatrix.x4: (rows kb..kb+7, cols 16ks..), (same rows, cols 16ks+8..), (rows kb+8.., 16ks..), (.., 16ks+8..)
            const int mi = lane >> 3;
            const uint32_t a0 = smem_addr(sK + (kb + (mi >> 1) * 8 + (lane & 7)) * kPitch + (mi & 1) * 16);
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                uint32_t r[4];
                ldmatrix_x4(a0 + ks * 32, r);
                mma_bf16(s[0], qa[ks], r[0], r[1]);
                mma_bf16(s[1], qa[ks], r[2], r[3]);
            }
        }
        // element (row g + 8 (j >> 1), tile row kb + 8 nb + 2t + (j & 1)) = s[nb][j]
        const long long row_base = r_begin + i * kTileRows + kb + 2 * t;
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nb = 0; nb < 2; ++nb) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const bool ok = row_base + 8 * nb + (j & 1) < r_end;
                s[nb][j] = ok ? s[nb][j] * c2 : -INFINITY;
                mx[j >> 1] = fmaxf(mx[j >> 1], s[nb][j]);
            }
        }
        uint32_t pa[4];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
            const float m_new = fmaxf(m[h], mx[h]);
            const float resc = m_new > -INFINITY ? exp2f(m[h] - m_new) : 1.f;       // m = -inf gives 0
            const float sub = m_new > -INFINITY ? m_new : 0.f;
            m[h] = m_new;
            z[h] *= resc;
#pragma unroll
            for (int nb = 0; nb < NB; ++nb) { o[nb][2 * h] *= resc; o[nb][2 * h + 1] *= resc; }
            const float p00 = exp2f(s[0][2 * h] - sub), p01 = exp2f(s[0][2 * h + 1] - sub);
            const float p10 = exp2f(s[1][2 * h] - sub), p11 = exp2f(s[1][2 * h + 1] - sub);
            z[h] += (p00 + p01) + (p10 + p11);
            pa[h] = pack2(p00, p01);                        // A fragment: a0/a1 = rows g/g+8 of tile rows kb+2t.., a2/a3 = kb+8+2t..
            pa[2 + h] = pack2(p10, p11);
        }
        {
            // matrices of one ldmatrix.x4.trans: (rows kb.., cols 16j..), (rows kb+8.., 16j..), (rows kb.., 16j+8..), (rows kb+8.., 16j+8..)
            const int mi = lane >> 3;
            const uint32_t a0 = smem_addr(sV + (kb + (mi & 1) * 8 + (lane & 7)) * kPitch + (mi >> 1) * 16);
#pragma unroll
            for (int j = 0; j < NB / 2; ++j) {
                uint32_t r[4];
                ldmatrix_x4_trans(a0 + j * 32, r);
                mma_bf16(o[2 * j], pa, r[0], r[1]);
                mma_bf16(o[2 * j + 1], pa, r[2], r[3]);
            }
        }
    }
    cp_async_wait<0>();
    __syncthreads();                                        // the tiles are done with: reuse the memory for the merge

    // merge the four warps: per query head (row) M, Z and the accumulator row
#pragma unroll
    for (int h = 0; h < 2; ++h) {
        z[h] += __shfl_xor_sync(0xffffffffu, z[h], 1);
        z[h] += __shfl_xor_sync(0xffffffffu, z[h], 2);
    }
    float* sm_o = reinterpret_cast<float*>(smem);           // [4 warps][16 rows][DH]
    float* sm_m = sm_o + 4 * 16 * DH;                       // [4][16]
    float* sm_z = sm_m + 4 * 16;
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) {
#pragma unroll
        for (int j = 0; j < 4; ++j)
            sm_o[((warp * 16) + g + (j >> 1) * 8) * DH + nb * 8 + 2 * t + (j & 1)] = o[nb][j];
    }
    if (t == 0) {
#pragma unroll
        for (int h = 0; h < 2; ++h) { sm_m[warp * 16 + g + 8 * h] = m[h]; sm_z[warp * 16 + g + 8 * h] = z[h]; }
    }
    __syncthreads();
    for (int idx = tid; idx < G * DH; idx += kThreads) {
        const int r = idx / DH, col = idx % DH;
        float M = -INFINITY;
#pragma unroll
        for (int w = 0; w < 4; ++w) M = fmaxf(M, sm_m[w * 16 + r]);
        float Z = 0.f, A = 0.f;
#pragma unroll
        for (int w = 0; w < 4; ++w) {
            const float f = M > -INFINITY ? exp2f(sm_m[w * 16 + r] - M) : 0.f;
            Z = fmaf(sm_z[w * 16 + r], f, Z);
            A = fmaf(sm_o[(w * 16 + r) * DH + col], f, A);
        }
        float* out = part0 + r * part_stride;
        out[2 + col] = A;
        if (col == 0) { out[0] = M; out[1] = Z; }
    }
}

template <int DH>
cudaError_t launch_t(const DecodePagedParams& p, cudaStream_t st) {
    const long long ctas = (long long)p.B * p.H_kv * p.total_chunks;
    if (ctas == 0) return cudaSuccess;
    const size_t smem = (size_t)kStages * 2 * kTileRows * (DH * 2 + 16);
    cudaError_t e = cudaFuncSetAttribute(decode_paged_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    decode_paged_kernel<DH><<<(unsigned)ctas, kThreads, smem, st>>>(p);
    return cudaGetLastError();
}

}  // namespace

cudaError_t launch_decode_paged(const DecodePagedParams& p, cudaStream_t st) {
    if (p.d == 128) return launch_t<128>(p, st);
    if (p.d == 64) return launch_t<64>(p, st);
    return cudaErrorNotSupported;
}

}  // namespace mka
