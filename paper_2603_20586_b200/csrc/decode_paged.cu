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
#include "tc_ptx.cuh"

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

// ---------------------------------------------------------------------------------------------------------------
// The same kernel fed by the copy engine.  Where every (page, KV head) block of a level is a box a tensor map can
// describe (pages of at least 8 rows, or a dense level), a fifth warp produces: lane i owns box i of every 64-row tile
// (a box = the rows of one page that fall into the tile), looks its page up and issues one TMA copy per 64-column
// panel of K and of V into 128-byte-swizzled tiles (a ring of three stages, one mbarrier pair per stage).  The four
// computing warps then issue no load instructions at all; ldmatrix reads the swizzled tiles without bank conflicts.
// Boxes that start past the chunk's last row are aimed at the chunk's first page (finite data, weights exactly 0);
// value rows past the last row inside the last box are cleared in shared memory before they are read, so that
// whatever a partly filled page holds there (NaN included) cannot reach the accumulator through 0 x NaN.
constexpr int kTmaThreads = 160;
constexpr int kTmaStages = 3;

struct PagedMaps {
    CUtensorMap k[3], v[3];
};

template <int DH>
__global__ void __launch_bounds__(kTmaThreads, 2) decode_paged_tma_kernel(const __grid_constant__ PagedMaps maps, const DecodePagedParams p) {
    constexpr int kPanels = DH / 64;
    constexpr int kPanelBytes = kTileRows * 128;            // [64 rows][64 bf16]
    constexpr int kTileBytes = kPanels * kPanelBytes;       // one of K or V
    constexpr int KS = DH / 16;
    constexpr int NB = DH / 8;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    __shared__ uint64_t full[kTmaStages], empty[kTmaStages];
    __shared__ WaitCtl ctl;
    __shared__ int s_pages[kSliceCap];

    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);
    const int g = lane >> 2, t = lane & 3;
    const int G = p.H / p.H_kv;
    long long chunk = blockIdx.x % p.total_chunks;
    const long long bk = blockIdx.x / p.total_chunks;
    const int b = (int)(bk / p.H_kv), kvh = (int)(bk % p.H_kv);
    const long long chunk_all = chunk;
    int lvl = 0;
    while (lvl < 2 && chunk >= p.n_chunks[lvl]) { chunk -= p.n_chunks[lvl]; ++lvl; }
    const PagedLevelDev L = p.L[lvl];
    long long n_b = L.rows ? (long long)L.rows[b] : L.n;
    n_b = n_b < 0 ? 0 : (n_b > L.n ? L.n : n_b);
    const long long r_begin = chunk * p.chunk_rows;
    const long long r_end = r_begin + p.chunk_rows < n_b ? r_begin + p.chunk_rows : n_b;
    const bool skip = p.gate[b * 3 + lvl] == 0.f || r_end <= r_begin;
    float* part0 = p.partial + (((long long)b * p.H + (long long)kvh * G) * p.total_chunks + chunk_all) * (DH + 2);
    const long long part_stride = p.total_chunks * (DH + 2);
    if (skip) {                                                                // nothing to read: empty partials
        for (int r = 0; r < G; ++r) {
            float* out = part0 + r * part_stride;
            for (int i = tid; i < DH + 2; i += kTmaThreads) out[i] = i == 0 ? -INFINITY : 0.f;
        }
        return;
    }
    if (tid == 0) {
        ctl.abort = 0;
        ctl.limit_ns = p.wait_limit_ns;
        for (int i = 0; i < kTmaStages; ++i) { mbar_init(&full[i], 1); mbar_init(&empty[i], 4); }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    const bool dense = L.table == nullptr;                  // one page per sequence: the page is the batch index
    const int shift = L.page_shift;
    const long long page_mask = ((long long)1 << shift) - 1;
    const long long page0 = r_begin >> shift;
    const int* table = dense ? nullptr : L.table + (long long)b * L.table_stride + (long long)kvh * L.table_head_stride + page0;
    const long long n_pages = ((r_end - 1) >> shift) - page0 + 1;
    const bool sliced = !dense && n_pages <= kSliceCap;
    if (sliced)
        for (int i = tid; i < (int)n_pages; i += kTmaThreads) s_pages[i] = table[i];
    __syncthreads();
    volatile WaitCtl* ctlp = &ctl;
    const long long n_tiles = (r_end - r_begin + kTileRows - 1) / kTileRows;

    if (warp == 4) {
        // ------------------------------------------------------------ producer
        const int box_rows = dense ? kTileRows : (int)(page_mask + 1 < kTileRows ? page_mask + 1 : kTileRows);
        const int boxes = kTileRows / box_rows;
        const bool mine = lane < boxes;
        bool ok = true;
        for (long long i = 0; i < n_tiles && ok; ++i) {
            const int st = (int)(i % kTmaStages);
            long long r0 = r_begin + i * kTileRows + (long long)lane * box_rows;
            if (r0 >= r_end) r0 = r_begin;                  // a box with no valid row re-reads the chunk's first box
            int page = b, in_row = (int)r0;
            if (!dense && mine) {
                const long long pi = (r0 >> shift) - page0;
                page = sliced ? s_pages[pi] : table[pi];
                in_row = (int)(r0 & page_mask);
            }
            if (!mbar_wait_warp(&empty[st], ((uint32_t)(i / kTmaStages) & 1u) ^ 1u, ctlp)) { ok = false; break; }
            if (lane == 0) mbar_expect_tx(&full[st], 2 * kTileBytes);
            __syncwarp();
            if (mine) {
                uint8_t* sK = smem + (size_t)st * 2 * kTileBytes + (size_t)lane * box_rows * 128;
#pragma unroll
                for (int pn = 0; pn < kPanels; ++pn) {
                    tma_load_4d(sK + pn * kPanelBytes, &maps.k[lvl], pn * 64, in_row, kvh, page, &full[st]);
                    tma_load_4d(sK + kTileBytes + pn * kPanelBytes, &maps.v[lvl], pn * 64, in_row, kvh, page, &full[st]);
                }
            }
        }
        // the shared memory must not be given up with a copy in flight: wait (bounded) for the stages still out
        const long long issued = n_tiles;
        if (ok)
            for (long long i = issued > kTmaStages ? issued - kTmaStages : 0; i < issued; ++i)
                mbar_wait_warp(&full[i % kTmaStages], (uint32_t)(i / kTmaStages) & 1u, ctlp);
        return;
    }

    // ---------------------------------------------------------------- computing warps
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
    const float c2 = p.scale * kLog2e;
    float m[2] = {-INFINITY, -INFINITY}, z[2] = {0.f, 0.f};
    float o[NB][4];
#pragma unroll
    for (int nb = 0; nb < NB; ++nb) { o[nb][0] = o[nb][1] = o[nb][2] = o[nb][3] = 0.f; }
    const int kb = warp * 16;                               // this warp's rows of a tile
    const int mi = lane >> 3, l7 = lane & 7;
    // ldmatrix row addresses inside a 128-byte-swizzled panel: row r, 16-byte chunk c sits at r * 128 + ((c ^ (r & 7)) << 4);
    // the rows a lane addresses have r & 7 = lane & 7
    const uint32_t k_row = (uint32_t)(kb + (mi >> 1) * 8 + l7) * 128u;
    const uint32_t v_row = (uint32_t)(kb + (mi & 1) * 8 + l7) * 128u;
    bool ok = true;
    for (long long i = 0; i < n_tiles; ++i) {
        const int st = (int)(i % kTmaStages);
        ok = mbar_wait_warp(&full[st], (uint32_t)(i / kTmaStages) & 1u, ctlp);
        if (!ok) break;
        uint8_t* sK = smem + (size_t)st * 2 * kTileBytes;
        uint8_t* sV = sK + kTileBytes;
        const long long tile_base = r_begin + i * kTileRows;
        if (tile_base + kb + 16 > r_end) {                  // clear this warp's value rows past the chunk's last row
            const int r_first = (int)max(0LL, r_end - tile_base - kb);       // first row (of the warp's 16) to clear
            for (int idx = lane; idx < (16 - r_first) * 8 * kPanels; idx += 32) {
                const int row = kb + r_first + idx / (8 * kPanels), rest = idx % (8 * kPanels);
                *reinterpret_cast<uint4*>(sV + (rest / 8) * kPanelBytes + row * 128 + (rest % 8) * 16) = make_uint4(0u, 0u, 0u, 0u);
            }
            __syncwarp();
        }
        float s[2][4];
#pragma unroll
        for (int nb = 0; nb < 2; ++nb) { s[nb][0] = s[nb][1] = s[nb][2] = s[nb][3] = 0.f; }
        {
            const uint32_t a0 = smem_addr(sK) + k_row;
#pragma unroll
            for (int ks = 0; ks < KS; ++ks) {
                const int c16 = ks * 2 + (mi & 1);          // 16-byte chunk of the row (0..15 at d = 128)
                uint32_t r[4];
                ldmatrix_x4(a0 + (uint32_t)((ks * 2) >> 3) * kPanelBytes + ((uint32_t)((c16 & 7) ^ l7) << 4), r);
                mma_bf16(s[0], qa[ks], r[0], r[1]);
                mma_bf16(s[1], qa[ks], r[2], r[3]);
            }
        }
        const long long row_base = tile_base + kb + 2 * t;
        float mx[2] = {-INFINITY, -INFINITY};
#pragma unroll
        for (int nb = 0; nb < 2; ++nb) {
#pragma unroll
            for (int j = 0; j < 4; ++j) {
                const bool in = row_base + 8 * nb + (j & 1) < r_end;
                s[nb][j] = in ? s[nb][j] * c2 : -INFINITY;
                mx[j >> 1] = fmaxf(mx[j >> 1], s[nb][j]);
            }
        }
        uint32_t pa[4];
#pragma unroll
        for (int h = 0; h < 2; ++h) {
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 1));
            mx[h] = fmaxf(mx[h], __shfl_xor_sync(0xffffffffu, mx[h], 2));
            const float m_new = fmaxf(m[h], mx[h]);
            const float resc = m_new > -INFINITY ? exp2f(m[h] - m_new) : 1.f;
            const float sub = m_new > -INFINITY ? m_new : 0.f;
            m[h] = m_new;
            z[h] *= resc;
#pragma unroll
            for (int nb = 0; nb < NB; ++nb) { o[nb][2 * h] *= resc; o[nb][2 * h + 1] *= resc; }
            const float p00 = exp2f(s[0][2 * h] - sub), p01 = exp2f(s[0][2 * h + 1] - sub);
            const float p10 = exp2f(s[1][2 * h] - sub), p11 = exp2f(s[1][2 * h + 1] - sub);
            z[h] += (p00 + p01) + (p10 + p11);
            pa[h] = pack2(p00, p01);
            pa[2 + h] = pack2(p10, p11);
        }
        {
            const uint32_t a0 = smem_addr(sV) + v_row;
#pragma unroll
            for (int j = 0; j < NB / 2; ++j) {
                const int c16 = j * 2 + (mi >> 1);
                uint32_t r[4];
                ldmatrix_x4_trans(a0 + (uint32_t)((j * 2) >> 3) * kPanelBytes + ((uint32_t)((c16 & 7) ^ l7) << 4), r);
                mma_bf16(o[2 * j], pa, r[0], r[1]);
                mma_bf16(o[2 * j + 1], pa, r[2], r[3]);
            }
        }
        __syncwarp();
        if (lane == 0) mbar_arrive(&empty[st]);             // this warp has read the stage
    }
    // The four warps meet at a named barrier that also carries their "no wait ran out" flags (the producer left already).
    {
        uint32_t out;
        asm volatile("{\n.reg .pred pi, po;\nsetp.ne.u32 pi, %1, 0;\nbar.red.and.pred po, 1, 128, pi;\nselp.u32 %0, 1, 0, po;\n}"
                     : "=r"(out) : "r"((uint32_t)ok) : "memory");
        if (!out) {
            if (tid == 0 && p.status) atomicExch(p.status, (unsigned int)MKA_ERR_TIMEOUT);
            return;
        }
    }
    // merge the four warps: per query head (row) M, Z and the accumulator row (the tiles are done with: reuse the memory)
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
    asm volatile("bar.sync 1, 128;" ::: "memory");
    for (int idx = tid; idx < G * DH; idx += 128) {
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

// The copy-engine form needs every non-empty level to be describable by a tensor map: a dense level, or pages of at
// least 8 rows; strides are multiples of 8 elements already.
template <int DH>
cudaError_t launch_tma(const DecodePagedParams& p, cudaStream_t st) {
    PagedMaps maps;
    for (int l = 0; l < 3; ++l) {
        const PagedLevelDev& L = p.L[l];
        bool made;
        if (L.n == 0) {                                     // never dereferenced: any valid descriptor will do
            made = true;
            if (l > 0) { maps.k[l] = maps.k[0]; maps.v[l] = maps.v[0]; }
            else memset(&maps.k[0], 0, sizeof(CUtensorMap)), memset(&maps.v[0], 0, sizeof(CUtensorMap));
            continue;
        }
        if (L.table == nullptr) {
            made = make_bf16_map(&maps.k[l], L.k, DH, L.n, p.H_kv, p.B, L.sn, L.sh, L.sp, kTileRows) &&
                   make_bf16_map(&maps.v[l], L.v, DH, L.n, p.H_kv, p.B, L.sn, L.sh, L.sp, kTileRows);
        } else {
            const int page_rows = 1 << L.page_shift;
            const int box = page_rows < kTileRows ? page_rows : kTileRows;
            // the pool's page count is not part of this call: the map claims the largest extent, the table bounds the reads
            const int pages = L.pool_pages > 0 && L.pool_pages < 0x7fffffffLL ? (int)L.pool_pages : 0x7fffffff;
            made = make_bf16_map(&maps.k[l], L.k, DH, page_rows, p.H_kv, pages, L.sn, L.sh, L.sp, box) &&
                   make_bf16_map(&maps.v[l], L.v, DH, page_rows, p.H_kv, pages, L.sn, L.sh, L.sp, box);
        }
        if (!made) return cudaErrorNotSupported;
    }
    // a level with n == 0 that comes first borrows the first real level's maps
    int first_real = -1;
    for (int l = 0; l < 3; ++l) if (p.L[l].n > 0) { first_real = l; break; }
    if (first_real < 0) return cudaSuccess;
    for (int l = 0; l < 3; ++l) if (p.L[l].n == 0) { maps.k[l] = maps.k[first_real]; maps.v[l] = maps.v[first_real]; }
    const long long ctas = (long long)p.B * p.H_kv * p.total_chunks;
    const size_t smem = (size_t)kTmaStages * 2 * kTileRows * DH * 2 + 1024;
    cudaError_t e = cudaFuncSetAttribute(decode_paged_tma_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    decode_paged_tma_kernel<DH><<<(unsigned)ctas, kTmaThreads, smem, st>>>(maps, p);
    return cudaGetLastError();
}

bool tma_eligible(const DecodePagedParams& p) {
    if (!tensor_map_encoder_available()) return false;
    for (int l = 0; l < 3; ++l) {
        const PagedLevelDev& L = p.L[l];
        if (L.n == 0) continue;
        if (L.table != nullptr && (L.page_shift < 3 || L.page_shift > 30)) return false;     // pages of 8 rows at least
        if (L.sn <= 0 || L.sn % 8 || L.sh % 8 || L.sp % 8 || L.sp < 0) return false;
        if (L.sp == 0 && (L.table != nullptr || p.B > 1)) return false;
        if (p.H_kv > 1 && L.sh <= 0) return false;
        if (L.n > 0x7fffffffLL) return false;
    }
    return true;
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
    if ((long long)p.B * p.H_kv * p.total_chunks == 0) return cudaSuccess;
    if (p.d != 128 && p.d != 64) return cudaErrorNotSupported;
    if (tma_eligible(p)) {
        const cudaError_t e = p.d == 128 ? launch_tma<128>(p, st) : launch_tma<64>(p, st);
        if (e != cudaErrorNotSupported) return e;           // a map could not be encoded: the first form takes any layout
    }
    return p.d == 128 ? launch_t<128>(p, st) : launch_t<64>(p, st);
}

}  // namespace mka
