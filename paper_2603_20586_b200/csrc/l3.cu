// L3 recall (Alg. 2 step 4, "L3 <- Retrieve(Q_h)"; the method section's vectorized hashing with chunk-based recall).
// The paper names the mechanism but not the hash.  Here a chunk is one page of the long-term key pool and its
// signature is a sign-random-projection code of the SUM of its keys; a query's code comes from the sum of the query
// heads that share the KV head; the R chunks whose codes agree with the query's in the most bits are recalled (ties
// to the earlier chunk) and listed in bank order as a page table for the paged decode.
// Code bits are decided by fp32 arithmetic, so its order is fixed: sums run row by row, a projection is one fmaf
// chain over the columns.
//   l3_index_kernel     HBM-bound: reads every key of the pool once, writes bits/8 bytes per (page, KV head)
//   l3_retrieve_kernel  one CTA per (sequence, KV head): query code, Hamming scores of the bank, R selection rounds
#include "common.cuh"

namespace mka {
namespace {

constexpr int kIdxThreads = 128;
constexpr int kIdxPairs = 32;                         // (page, head) pairs per batch of a CTA: one per lane in the projections
constexpr int kIdxBitsPerWarp = 16;                   // code bits one warp works out per pass

struct L3IndexParams {
    const __nv_bfloat16* k;
    const float* proj;       // [bits, d]
    unsigned int* codes;     // [pages, H_kv, bits / 32]
    long long n_pages, sp, sh, sn;
    int H_kv, page_rows, d, bits;
};

// Dynamic shared memory: projT [d][bits + 4] floats (16 consecutive bits of one column are one broadcast read), then
// s [kIdxPairs][d + 1] floats (the key sums; the odd pitch keeps the lanes of a warp on different banks).
// A batch = 32 (page, head) pairs.  Loading: 16 threads cover one 256-byte row, a thread sums its eight columns row by
// row.  Projections: lane = pair, warp = 16 bits; column i costs one read of s, four broadcast reads of projT and 16
// fmaf, so the arithmetic, not shared memory, is what the projections wait for.
template <int DH>
__global__ void __launch_bounds__(kIdxThreads, 4) l3_index_kernel(const L3IndexParams p) {
    extern __shared__ __align__(16) float sm[];
    const int ppitch = p.bits + 4;                             // floats between columns of projT (keeps the fill off one bank)
    float* projT = sm;
    float* s = sm + (size_t)DH * ppitch;
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    constexpr int pitch = DH + 1;
    for (int e = tid; e < DH * p.bits; e += kIdxThreads) {     // e = j * d + i: coalesced reads of proj
        const int j = e / DH, i = e % DH;
        projT[i * ppitch + j] = p.proj[e];
    }
    constexpr int vecs = DH / 8;                               // 16-byte pieces of a row: 16 (d = 128) or 8 (d = 64)
    constexpr int items = kIdxPairs * vecs;                    // (pair, piece) items of a batch
    constexpr int kPerThread = items / kIdxThreads;            // 4 or 2: taken two at a time, 16 loads in flight
    const long long pairs = p.n_pages * p.H_kv;
    const int words = p.bits / 32;
    unsigned short* codes16 = reinterpret_cast<unsigned short*>(p.codes);
    for (long long base = (long long)blockIdx.x * kIdxPairs; base < pairs; base += (long long)gridDim.x * kIdxPairs) {
        __syncthreads();                                       // projT is there; the previous batch is done with s
        // ---- sums of the pages' keys, row by row
#pragma unroll
        for (int k0 = 0; k0 < kPerThread; k0 += 2) {
            float acc[2][8];
            const __nv_bfloat16* src[2];
            bool live[2];
            int slot[2], piece[2];
#pragma unroll
            for (int q = 0; q < 2; ++q) {
                const int it = tid + (k0 + q) * kIdxThreads;
                slot[q] = it / vecs; piece[q] = it % vecs;
                const long long pair = base + slot[q];
                live[q] = pair < pairs;
                const long long pc = live[q] ? pair : 0;
                src[q] = p.k + (pc / p.H_kv) * p.sp + (pc % p.H_kv) * p.sh + piece[q] * 8;
#pragma unroll
                for (int i = 0; i < 8; ++i) acc[q][i] = 0.f;
            }
            for (int r0 = 0; r0 < p.page_rows; r0 += 8) {
                uint4 u[2][8];
#pragma unroll
                for (int q = 0; q < 2; ++q)
#pragma unroll
                    for (int r = 0; r < 8; ++r)
                        u[q][r] = (live[q] && r0 + r < p.page_rows)
                                      ? __ldg(reinterpret_cast<const uint4*>(src[q] + (long long)(r0 + r) * p.sn))
                                      : make_uint4(0u, 0u, 0u, 0u);
#pragma unroll
                for (int q = 0; q < 2; ++q)
#pragma unroll
                    for (int r = 0; r < 8; ++r) {
                        if (r0 + r < p.page_rows) {                // rows past the page add nothing, not even +0
                            const uint32_t w[4] = {u[q][r].x, u[q][r].y, u[q][r].z, u[q][r].w};
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                acc[q][2 * i] = acc[q][2 * i] + __uint_as_float(w[i] << 16);
                                acc[q][2 * i + 1] = acc[q][2 * i + 1] + __uint_as_float(w[i] & 0xffff0000u);
                            }
                        }
                    }
            }
#pragma unroll
            for (int q = 0; q < 2; ++q)
#pragma unroll
                for (int i = 0; i < 8; ++i) s[slot[q] * pitch + piece[q] * 8 + i] = acc[q][i];
        }
        __syncthreads();
        // ---- projections: one fmaf chain per (pair, bit) over the columns 0..d-1
        const long long pair = base + lane;
        const float* sv = s + lane * pitch;
        for (int j0 = warp * kIdxBitsPerWarp; j0 < p.bits; j0 += (kIdxThreads / 32) * kIdxBitsPerWarp) {
            // two chains per instruction (fma.rn.f32x2: each half is the same correctly rounded fma as fmaf)
            unsigned long long a2[kIdxBitsPerWarp / 2];
#pragma unroll
            for (int j = 0; j < kIdxBitsPerWarp / 2; ++j) a2[j] = 0ull;          // two +0.f
            const float* pj = projT + j0;
            for (int i = 0; i < DH; ++i) {
                const float x = sv[i];
                unsigned long long x2;
                asm("mov.b64 %0, {%1, %1};" : "=l"(x2) : "f"(x));
#pragma unroll
                for (int v = 0; v < kIdxBitsPerWarp / 4; ++v) {
                    const ulonglong2 pr = *reinterpret_cast<const ulonglong2*>(pj + (size_t)i * ppitch + 4 * v);   // bits 4v..4v+3 of column i
                    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(a2[2 * v]) : "l"(pr.x), "l"(x2));
                    asm("fma.rn.f32x2 %0, %1, %2, %0;" : "+l"(a2[2 * v + 1]) : "l"(pr.y), "l"(x2));
                }
            }
            unsigned half = 0u;
#pragma unroll
            for (int j = 0; j < kIdxBitsPerWarp / 2; ++j) {
                float lo, hi;
                asm("mov.b64 {%0, %1}, %2;" : "=f"(lo), "=f"(hi) : "l"(a2[j]));
                half |= (lo >= 0.f ? 1u : 0u) << (2 * j);
                half |= (hi >= 0.f ? 1u : 0u) << (2 * j + 1);
            }
            // bits j0..j0+15 are one 16-bit half of word j0 / 32 (low half first)
            if (pair < pairs) codes16[(pair * words) * 2 + j0 / 16] = (unsigned short)half;
        }
    }
}

struct L3RetrieveParams {
    const __nv_bfloat16* q;       // [B, H, d]
    const float* proj;            // [bits, d]
    const unsigned int* codes;    // [pages, H_kv, words]
    const int* bank;              // [B, bank_stride]
    const int* bank_len;          // [B]
    int* table;                   // [B, H_kv, R]
    int* n_sel;                   // [B] or null
    int* rows;                    // [B] or null: n_sel * page_rows
    long long bank_stride;
    int B, H, H_kv, d, bits, R, page_rows, max_bank;
};

constexpr int kRetThreads = 1024;
constexpr int kMaxR = 64;
constexpr unsigned short kTaken = 0xffffu;

// dynamic shared memory: unsigned short score[max_bank]
__global__ void __launch_bounds__(kRetThreads) l3_retrieve_kernel(const L3RetrieveParams p) {
    extern __shared__ __align__(16) unsigned short score[];
    __shared__ float qs[256];
    __shared__ unsigned int qcode[8];
    __shared__ unsigned long long red[kRetThreads / 32];
    __shared__ int sel[kMaxR];
    const int tid = threadIdx.x, lane = tid & 31, warp = tid >> 5;
    const int b = blockIdx.x / p.H_kv, kvh = blockIdx.x % p.H_kv;
    const int G = p.H / p.H_kv, words = p.bits / 32;
    // query of the KV head: the group's heads summed in head order, fp32
    if (tid < p.d) {
        const __nv_bfloat16* q0 = p.q + ((long long)b * p.H + (long long)kvh * G) * p.d + tid;
        float acc = 0.f;
        for (int g = 0; g < G; ++g) acc = acc + __bfloat162float(q0[(long long)g * p.d]);
        qs[tid] = acc;
    }
    if (tid < 8) qcode[tid] = 0u;
    __syncthreads();
    if (tid < p.bits) {
        const float* pr = p.proj + (long long)tid * p.d;
        float acc = 0.f;
        for (int i = 0; i < p.d; ++i) acc = fmaf(pr[i], qs[i], acc);
        if (acc >= 0.f) atomicOr(&qcode[tid >> 5], 1u << (tid & 31));
    }
    __syncthreads();
    int n = p.bank_len[b];
    n = n < 0 ? 0 : (n > p.max_bank ? p.max_bank : n);
    const int* bank = p.bank + (long long)b * p.bank_stride;
    // eight chunks per thread at a time: the page numbers first, then all their code words, so that the two dependent
    // gathers cost two round trips per eight chunks and not two per chunk
    for (int c0 = tid; c0 < n; c0 += 8 * kRetThreads) {
        int page[8];
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            const int c = c0 + u * kRetThreads;
            page[u] = c < n ? bank[c] : 0;
        }
        if (words == 2) {                                      // 64-bit codes: one 8-byte load per chunk
            uint2 w[8];
#pragma unroll
            for (int u = 0; u < 8; ++u)
                w[u] = __ldg(reinterpret_cast<const uint2*>(p.codes + ((long long)page[u] * p.H_kv + kvh) * 2));
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int c = c0 + u * kRetThreads;
                if (c < n) score[c] = (unsigned short)(p.bits - __popc(w[u].x ^ qcode[0]) - __popc(w[u].y ^ qcode[1]));
            }
        } else {
#pragma unroll
            for (int u = 0; u < 8; ++u) {
                const int c = c0 + u * kRetThreads;
                if (c >= n) continue;
                const unsigned int* code = p.codes + ((long long)page[u] * p.H_kv + kvh) * words;
                int dist = 0;
                for (int w = 0; w < words; ++w) dist += __popc(__ldg(code + w) ^ qcode[w]);
                score[c] = (unsigned short)(p.bits - dist);    // agreement: 0..bits (<= 256)
            }
        }
    }
    __syncthreads();
    const int k = p.R < n ? p.R : n;
    for (int r = 0; r < k; ++r) {
        // key = agreement in the high half, inverted position in the low half: the maximum is the best score, earliest chunk
        unsigned long long best = 0ull;
        for (int c = tid; c < n; c += kRetThreads) {
            const unsigned short sc = score[c];
            if (sc == kTaken) continue;
            const unsigned long long key = ((unsigned long long)(sc + 1u) << 32) | (unsigned)(0x7fffffff - c);
            best = key > best ? key : best;
        }
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) {
            const unsigned long long other = __shfl_xor_sync(0xffffffffu, best, o);
            best = other > best ? other : best;
        }
        if (lane == 0) red[warp] = best;
        __syncthreads();
        if (tid == 0) {
            unsigned long long m = red[0];
            for (int w = 1; w < kRetThreads / 32; ++w) m = red[w] > m ? red[w] : m;
            const int c = 0x7fffffff - (int)(m & 0xffffffffu);
            sel[r] = c;
            score[c] = kTaken;
        }
        __syncthreads();
    }
    if (tid == 0) {
        for (int i = 1; i < k; ++i) {                           // bank (time) order
            const int v = sel[i];
            int j = i - 1;
            while (j >= 0 && sel[j] > v) { sel[j + 1] = sel[j]; --j; }
            sel[j + 1] = v;
        }
        int* out = p.table + ((long long)b * p.H_kv + kvh) * p.R;
        for (int i = 0; i < p.R; ++i) out[i] = i < k ? bank[sel[i]] : 0;
        if (kvh == 0) {
            if (p.n_sel) p.n_sel[b] = k;
            if (p.rows) p.rows[b] = k * p.page_rows;
        }
    }
}

}  // namespace

cudaError_t launch_l3_index(const void* k, long long n_pages, int H_kv, int page_rows, int d, long long sp, long long sh,
                            long long sn, const float* proj, int bits, unsigned int* codes, cudaStream_t st) {
    if (n_pages == 0 || H_kv == 0) return cudaSuccess;
    L3IndexParams p;
    p.k = static_cast<const __nv_bfloat16*>(k); p.proj = proj; p.codes = codes;
    p.n_pages = n_pages; p.sp = sp; p.sh = sh; p.sn = sn; p.H_kv = H_kv; p.page_rows = page_rows; p.d = d; p.bits = bits;
    const size_t smem = ((size_t)d * (bits + 4) + (size_t)kIdxPairs * (d + 1)) * sizeof(float);
    auto kern = d == 128 ? l3_index_kernel<128> : l3_index_kernel<64>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    const long long batches = (n_pages * H_kv + kIdxPairs - 1) / kIdxPairs;
    const long long per_sm = smem > 110 * 1024 ? 1 : (smem > 72 * 1024 ? 2 : (smem > 54 * 1024 ? 3 : 4));
    const long long resident = 148LL * per_sm;
    // persistent CTAs: every CTA transposes the projection into shared memory once and then walks its batches
    // (the grid is shrunk so that all CTAs get the same number of batches)
    const long long per_cta = (batches + resident - 1) / resident;
    const long long grid = (batches + per_cta - 1) / per_cta;
    kern<<<(unsigned)grid, kIdxThreads, smem, st>>>(p);
    return cudaGetLastError();
}

cudaError_t launch_l3_retrieve(const void* q, int B, int H, int H_kv, int d, const float* proj, int bits,
                               const unsigned int* codes, const int* bank, const int* bank_len, long long bank_stride,
                               int max_bank, int R, int page_rows, int* table, int* n_sel, int* rows, cudaStream_t st) {
    if (B == 0 || H_kv == 0) return cudaSuccess;
    L3RetrieveParams p;
    p.q = static_cast<const __nv_bfloat16*>(q); p.proj = proj; p.codes = codes; p.bank = bank; p.bank_len = bank_len;
    p.table = table; p.n_sel = n_sel; p.rows = rows; p.bank_stride = bank_stride;
    p.B = B; p.H = H; p.H_kv = H_kv; p.d = d; p.bits = bits; p.R = R; p.page_rows = page_rows; p.max_bank = max_bank;
    const size_t smem = ((size_t)(max_bank > 0 ? max_bank : 1) * sizeof(unsigned short) + 15) / 16 * 16;
    cudaError_t e = cudaFuncSetAttribute(l3_retrieve_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)smem);
    if (e != cudaSuccess) return e;
    l3_retrieve_kernel<<<(unsigned)(B * H_kv), kRetThreads, smem, st>>>(p);
    return cudaGetLastError();
}

}  // namespace mka
