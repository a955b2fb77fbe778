// Tensor-core backward of Eq. 5 for bf16 on sm_100a: TMA -> shared memory -> tcgen05.mma -> TMEM.
//
// The paper prints no backward; this one follows from differentiating Eq. 5.  With
//   p = lambda_{t,l} exp(s - LSE_t) on the visible set,  dP = dO_t . v_{l,j},  D_t = dO_t . O_t,
//   dS = p (dP - D_t):
//     dV_{l,j} = sum_t p dO_t      dK_{l,j} = tau sum_t dS q_t      dQ_t = tau sum_{l,j} dS k_{l,j}
//     G_{t,l}  = sum_{j in l} dS   (gradient of the router logit of level l, per head)
//
// Three launches, each deterministic (every output element has one owner, fixed summation order):
//   bwd_prep_kernel    per (b,h,t): D_t and, per level, the exponent bias log2(lambda) - LSE log2(e)
//   bwd_dq_tc_kernel   CTA = 128 query rows of one (b,h); streams the level-ordered list of 128-row
//                      key tiles (L1 window, L2 prefix, L3 slots) exactly like the forward:
//                      S = Q K^T, dP = dO V^T (128x128 each), dS -> TMEM (bf16), dQ += dS K.
//   bwd_dkv_tc_kernel  CTA = 128 key rows of one level of one (b,h); streams the 128-row query
//                      tiles that can see them: S^T = K Q^T, dP^T = V dO^T, P^T and dS^T -> TMEM
//                      (bf16), dV += P^T dO, dK += dS^T Q.
// Both kernels recompute the scores (7 matrix products per visible tile pair instead of 5) in exchange
// for needing no atomics and no cross-CTA reduction.
//
// In the dK/dV kernel the per-query terms vary along the COLUMNS of the transposed tiles, where a thread would need 64
// biases and 64 D_t per tile from shared memory (which the tensor pipe saturates).  They enter through the tensor pipe
// instead: both score products get a ninth K-step whose key-side operand is ones and whose query-side operand holds
// bias_t / scale (for S^T) or -D_t (for dP^T), each split into three bf16 terms, so S^T + bias / scale and dP^T - D arrive
// in TMEM ready-made.  The producing warp writes those 4 KB operand slabs (no swizzle) from the statistics of the prep
// kernel, fetched one tile ahead.  Q tiles and dO tiles travel in rings of their own: dO(e) is free again after dV(e),
// Q(e) only after dK(e), and Q(e+1) is what the next score product waits for.  Half of the exponentials of that kernel
// run as a cubic on the FMA pipe (exp2_pair_fma).
//
// Warp roles (320 threads): warps 0-7 are the element-wise ("softmax") threads: thread i of either
// warpgroup owns TMEM lane i & 127 (a query row in the dQ kernel, a key row in the dK/dV kernel);
// warpgroup 0 takes columns 0-63 of a tile and warpgroup 1 columns 64-127.  Their work on a tile has
// two phases so that it overlaps the tensor pipe: phase 1 needs only S (p = 2^(s*scale + bias), kept in
// registers) and runs while dP is still being multiplied; phase 2 reads dP, forms dS = p (dP - D) and
// writes it (bf16) over the columns of dP it has just read.  Warp 8 issues the TMA loads (lane 0);
// warp 9 issues every tcgen05.mma, running its loop converged with one elected lane issuing.
// TMEM (512 columns), dQ kernel: S ping [0,128), S pong [128,256), dP/dS [256,384), dQ [384,384+d).
//                     dK/dV kernel: S^T/P^T [0,128), dP^T/dS^T [128,256), dK [256,256+d), dV [256+d,256+2d).
// Every mbarrier wait is bounded; on expiry the CTA raises a flag, drains and reports MKA_ERR_TIMEOUT.
#include "tc_ptx.cuh"

namespace mka {
namespace {

constexpr int kThreads = 320;
constexpr int kProducerWarp = 8, kMmaWarp = 9;
constexpr int kBlk = 128;                             // rows of every tile
constexpr uint32_t kPanel = 128 * 128;                // bytes of a [128 rows][64 bf16] panel
constexpr int kMaxStages = 4;

struct BwdMaps {
    CUtensorMap q, dO;
    CUtensorMap k[3], v[3];
};

struct BwdTcParams {
    __nv_bfloat16* dQ;
    const float* statD;       // [B*H, Tpad]  D_t = dO_t . O_t
    const float* statB[3];    // per level: [B*H, Tpad]  log2(lambda_{t,l}) - LSE_t log2(e)  (-inf on padding rows)
    float* Gpart;             // [B, H, T, 3]
    LevelGradDev dL[3];
    long long n[3];
    int B, H, T, Tpad;
    int kv_group;             // query heads per KV head: K, V, dK, dV hold H / kv_group heads
    int window, q_offset;
    float scale, scale_log2;
    int kv_tiles[3];          // 128-row key tiles per level
    unsigned int* status;
    unsigned long long wait_limit_ns;
    int test_stall;           // test hook: the dK/dV kernel's loader leaves out the last query tile of every CTA
};

// v as a sum of three bf16 terms (exact to 2^-25 |v|) in the first three of eight bf16 slots of a 16-byte core-matrix row;
// an infinite v (the bias of a padding row or of a level the gate closes) stays one infinite term.
__device__ __forceinline__ uint4 split3_bf16(float v) {
    if (!(fabsf(v) <= 3.0e38f)) return make_uint4(pack_bf16(v, 0.f), 0u, 0u, 0u);
    const float t0 = __bfloat162float(__float2bfloat16_rn(v));
    const float r1 = v - t0;
    const float t1 = __bfloat162float(__float2bfloat16_rn(r1));
    return make_uint4(pack_bf16(t0, t1), pack_bf16(r1 - t1, 0.f), 0u, 0u);
}

// 2^x for two arguments x <= 0 on the FMA pipe: x is clamped to -127 and split into n = round(x) and f = x - n in
// [-1/2, 1/2] by adding and subtracting 1.5 * 2^23 (the sum's low mantissa bits are n); 2^f is a cubic with constant term
// exactly 1 (coefficients fitted for the smallest maximum relative error, 1.0e-4, a twentieth of the rounding step of
// the bf16 value it becomes); n is added to the exponent field.  x <= -127 gives exactly 0, as ex2 does for -inf.
__device__ __forceinline__ void exp2_pair_fma(float x0, float x1, float& p0, float& p1) {
    const float kMagic = 12582912.f;
    const uint64_t x = pack2(fmaxf(x0, -127.f), fmaxf(x1, -127.f));
    const uint64_t t = add2(x, pack2(kMagic, kMagic));
    const uint64_t n = add2(t, pack2(-kMagic, -kMagic));
    const uint64_t f = fma2(n, pack2(-1.f, -1.f), x);
    uint64_t r = fma2(pack2(0.05500893f, 0.05500893f), f, pack2(0.24221095f, 0.24221095f));
    r = fma2(r, f, pack2(0.69328290f, 0.69328290f));
    r = fma2(r, f, pack2(1.f, 1.f));
    float r0, r1, t0, t1;
    unpack2(r, r0, r1);
    unpack2(t, t0, t1);
    p0 = __uint_as_float(__float_as_uint(r0) + (__float_as_uint(t0) << 23));
    p1 = __uint_as_float(__float_as_uint(r1) + (__float_as_uint(t1) << 23));
}

template <int DH>
struct BCfg {
    static constexpr int kPanels = DH / 64;
    static constexpr uint32_t kTile = kPanels * kPanel;       // a 128-row tile
    static constexpr int kStages = DH == 128 ? 2 : 4;         // also keeps the CTA above half of shared memory
    // dK/dV kernel: the per-query terms enter the two score products as one more K-step (see kAugBytes below)
    static constexpr uint32_t kAugBytes = kBlk * 16 * 2;              // a [128 rows][16] bf16 operand slab without swizzle
    static constexpr int kStagesK = DH == 128 ? 3 : 4;        // K ring of the dQ kernel: K(e) stays in use until dQ(e), two tiles after it is first read
    static constexpr uint32_t kSmemDq = 2 * kTile + (kStages + kStagesK) * kTile + 1024;
    static constexpr uint32_t kSmemDkv = 2 * kTile + kStages * (2 * kTile + 2 * kAugBytes) + kAugBytes + 1024;
    // instruction descriptors: fp32 accumulate, bf16 x bf16, M = 128
    static constexpr uint32_t kIdescS = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kBlk >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
    static constexpr uint32_t kIdescAcc = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(DH >> 3) << 17) | ((uint32_t)(128 >> 4) << 24);
};

struct BwdBarriers {
    uint64_t fixed_full;                                  // the CTA's own (non-streamed) tiles
    uint64_t a_full[kMaxStages], a_empty[kMaxStages];     // streamed ring (dQ kernel: K tiles; dK/dV kernel: Q tiles + bias slabs)
    uint64_t b_full[kMaxStages], b_empty[kMaxStages];     // second streamed ring (dQ kernel: V tiles; dK/dV kernel: dO tiles + D slabs)
    uint64_t s_full[2];                                   // S landed in TMEM (dQ kernel: ping, pong)
    uint64_t dp_full;                                     // dP landed in TMEM
    uint64_t p_part[2];                                   // phase 1 (dK/dV kernel): the first / second 32 columns of every thread's P^T are written
    uint64_t ds_part[2];                                  // phase 2: the same for dS
    uint64_t acc_done;
};

__device__ __forceinline__ void softmax_group_sync() { asm volatile("bar.sync 1, 256;" ::: "memory"); }

// ------------------------------------------------------------------------------------------ prep
// D = dO . O and the three exponent biases of every padded row.  DH / 8 lanes share a row (one 16-byte load of O and
// one of dO each), a warp covers 2 or 4 rows per pass and a thread works on four passes at once, so eight loads are
// in flight per thread.  Padding rows (t >= T) get a bias of -inf so that a streamed sub-tile may run past the last
// query without a mask.
template <int DH>
__global__ void __launch_bounds__(256) bwd_prep_kernel(const __nv_bfloat16* __restrict__ O, const __nv_bfloat16* __restrict__ dO,
                                                       const float* __restrict__ LSE, const float* __restrict__ gate, int H,
                                                       int T, int Tpad, long long rows_pad, float* __restrict__ sD,
                                                       float* __restrict__ b0, float* __restrict__ b1, float* __restrict__ b2) {
    constexpr int LPR = DH / 8;                            // lanes per row: 16 or 8
    constexpr int RPW = 32 / LPR;                          // rows per warp and pass
    constexpr int kPasses = 4;
    const int lane = threadIdx.x & 31, sub = lane % LPR, grp = lane / LPR;
    const long long warp_row0 = ((long long)blockIdx.x * 8 + (threadIdx.x >> 5)) * (RPW * kPasses);
    uint4 a[kPasses], g[kPasses];
    long long rr[kPasses];
    bool in[kPasses];
#pragma unroll
    for (int u = 0; u < kPasses; ++u) {
        rr[u] = warp_row0 + u * RPW + grp;
        const long long bh = rr[u] / Tpad;
        const int t = (int)(rr[u] % Tpad);
        in[u] = rr[u] < rows_pad && t < T;
        a[u] = g[u] = make_uint4(0u, 0u, 0u, 0u);
        if (in[u]) {
            const long long off = (bh * T + t) * DH + sub * 8;
            a[u] = __ldg(reinterpret_cast<const uint4*>(O + off));
            g[u] = __ldg(reinterpret_cast<const uint4*>(dO + off));
        }
    }
#pragma unroll
    for (int u = 0; u < kPasses; ++u) {
        const uint32_t aw[4] = {a[u].x, a[u].y, a[u].z, a[u].w}, gw[4] = {g[u].x, g[u].y, g[u].z, g[u].w};
        float s = 0.f;
#pragma unroll
        for (int i = 0; i < 4; ++i) {
            s = fmaf(__uint_as_float(aw[i] << 16), __uint_as_float(gw[i] << 16), s);
            s = fmaf(__uint_as_float(aw[i] & 0xffff0000u), __uint_as_float(gw[i] & 0xffff0000u), s);
        }
#pragma unroll
        for (int o = LPR / 2; o > 0; o >>= 1) s += __shfl_xor_sync(0xffffffffu, s, o);
        if (sub == 0 && rr[u] < rows_pad) {
            float o0 = -INFINITY, o1 = -INFINITY, o2 = -INFINITY;
            if (in[u]) {
                const long long bh = rr[u] / Tpad;
                const int t = (int)(rr[u] % Tpad);
                const float lse = LSE[bh * T + t];
                const float* gt = gate + ((bh / H) * T + t) * 3;
                const bool live = lse > -INFINITY;
                const float l2 = lse * kLog2e;
                o0 = (live && gt[0] > 0.f) ? log2f(gt[0]) - l2 : -INFINITY;
                o1 = (live && gt[1] > 0.f) ? log2f(gt[1]) - l2 : -INFINITY;
                o2 = (live && gt[2] > 0.f) ? log2f(gt[2]) - l2 : -INFINITY;
            }
            sD[rr[u]] = in[u] ? s : 0.f;
            b0[rr[u]] = o0; b1[rr[u]] = o1; b2[rr[u]] = o2;
        }
    }
}

// Key tile range [first, end) (128-row units) of query rows [r0, r1] on one level.
__device__ __forceinline__ void key_tile_range(int level, long long r0, long long r1, int q_offset, int window, long long n,
                                               int& first, int& end) {
    long long lo_f, hi_f, lo_l, hi_l;
    visible_range(level, r0 + q_offset, window, n, 0, lo_f, hi_f);
    visible_range(level, r1 + q_offset, window, n, 0, lo_l, hi_l);
    const long long hi = hi_l > hi_f ? hi_l : hi_f;
    if (hi <= lo_f) { first = end = 0; return; }
    first = (int)(lo_f / kBlk);
    end = (int)((hi + kBlk - 1) / kBlk);
}

__device__ __forceinline__ void store_row_bf16(__nv_bfloat16* dst, const uint32_t (&o)[32], float mul) {
#pragma unroll
    for (int i = 0; i < 32; i += 8) {
        uint4 v;
        v.x = pack_bf16(__uint_as_float(o[i]) * mul, __uint_as_float(o[i + 1]) * mul);
        v.y = pack_bf16(__uint_as_float(o[i + 2]) * mul, __uint_as_float(o[i + 3]) * mul);
        v.z = pack_bf16(__uint_as_float(o[i + 4]) * mul, __uint_as_float(o[i + 5]) * mul);
        v.w = pack_bf16(__uint_as_float(o[i + 6]) * mul, __uint_as_float(o[i + 7]) * mul);
        *reinterpret_cast<uint4*>(dst + i) = v;
    }
}

// A-operand column (32-bit TMEM columns) of K-step k of a 128-wide bf16 row that the two warpgroups wrote
// as two packed halves: keys 0-63 at columns [0,32), keys 64-127 at columns [64,96) of the region.
__device__ __forceinline__ uint32_t packed_half_col(int k) { return (uint32_t)((k >> 2) * 64 + (k & 3) * 8); }

// ------------------------------------------------------------------------------------------ dQ
template <int DH>
__global__ void __launch_bounds__(kThreads, 1) bwd_dq_tc_kernel(const __grid_constant__ BwdMaps maps, const BwdTcParams p) {
    using C = BCfg<DH>;
    constexpr uint32_t kColS = 0, kColDP = 256, kColAcc = 384;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* sQ = smem;
    uint8_t* sdO = sQ + C::kTile;
    uint8_t* sK = sdO + C::kTile;                         // kStagesK tiles
    uint8_t* sV = sK + C::kStagesK * C::kTile;            // kStages tiles
    float (*gsm)[6] = reinterpret_cast<float (*)[6]>(sQ); // epilogue scratch; Q is dead once the last S product has completed
    __shared__ BwdBarriers bar;
    __shared__ uint32_t tmem_base_slot;
    __shared__ WaitCtl wait_ctl;

    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);   // tid >> 5, but provably warp-uniform for the compiler
    const int b = blockIdx.z, h = blockIdx.y;
    const long long bh = (long long)b * p.H + h;
    const int qtile = gridDim.x - 1 - blockIdx.x;          // latest (heaviest) rows first
    const long long m0 = (long long)qtile * kBlk;
    const long long m_last = (m0 + kBlk - 1 < p.T - 1) ? m0 + kBlk - 1 : p.T - 1;

    if (tid == 0) {
        wait_ctl.abort = 0;
        wait_ctl.limit_ns = p.wait_limit_ns;
        mbar_init(&bar.fixed_full, 1);
        for (int s = 0; s < kMaxStages; ++s) {
            mbar_init(&bar.a_full[s], 1); mbar_init(&bar.a_empty[s], 1);
            mbar_init(&bar.b_full[s], 1); mbar_init(&bar.b_empty[s], 1);
        }
        mbar_init(&bar.s_full[0], 1); mbar_init(&bar.s_full[1], 1);
        mbar_init(&bar.dp_full, 1);
        for (int i = 0; i < 2; ++i) { mbar_init(&bar.p_part[i], 8); mbar_init(&bar.ds_part[i], 8); }   // 8 = one arrival per element-wise warp
        mbar_init(&bar.acc_done, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_slot;
    volatile WaitCtl* abortp = &wait_ctl;

    int first[3], end[3];
#pragma unroll
    for (int l = 0; l < 3; ++l) {
        if (p.n[l] > 0) key_tile_range(l, m0, m_last, p.q_offset, p.window, p.n[l], first[l], end[l]);
        else first[l] = end[l] = 0;
    }
    const int E = (end[0] - first[0]) + (end[1] - first[1]) + (end[2] - first[2]);

    if (warp == kProducerWarp) {
        if (lane == 0) {
            mbar_expect_tx(&bar.fixed_full, 2 * C::kTile);
#pragma unroll
            for (int pn = 0; pn < C::kPanels; ++pn) {
                tma_load_4d(sQ + pn * kPanel, &maps.q, pn * 64, (int)m0, h, b, &bar.fixed_full);
                tma_load_4d(sdO + pn * kPanel, &maps.dO, pn * 64, (int)m0, h, b, &bar.fixed_full);
            }
            int issued_k = 0, issued_v = 0;
            bool ok = true;
            for (int l = 0; l < 3 && ok; ++l) {
                for (int kt = first[l]; kt < end[l]; ++kt) {
                    const int s = issued_k % C::kStagesK, sv = issued_k % C::kStages;
                    const uint32_t ph = (uint32_t)(issued_k / C::kStagesK) & 1u, phv = (uint32_t)(issued_k / C::kStages) & 1u;
                    if (!mbar_wait(&bar.a_empty[s], ph ^ 1u, abortp)) { ok = false; break; }
                    mbar_expect_tx(&bar.a_full[s], C::kTile);
#pragma unroll
                    for (int pn = 0; pn < C::kPanels; ++pn)
                        tma_load_4d(sK + s * C::kTile + pn * kPanel, &maps.k[l], pn * 64, kt * kBlk, h / p.kv_group, b, &bar.a_full[s]);
                    ++issued_k;
                    if (!mbar_wait(&bar.b_empty[sv], phv ^ 1u, abortp)) { ok = false; break; }
                    mbar_expect_tx(&bar.b_full[sv], C::kTile);
#pragma unroll
                    for (int pn = 0; pn < C::kPanels; ++pn)
                        tma_load_4d(sV + sv * C::kTile + pn * kPanel, &maps.v[l], pn * 64, kt * kBlk, h / p.kv_group, b, &bar.b_full[sv]);
                    ++issued_v;
                }
            }
            // every copy issued above must have landed before the shared memory can be given up
            mbar_wait(&bar.fixed_full, 0, abortp);
            for (int i = issued_k > C::kStagesK ? issued_k - C::kStagesK : 0; i < issued_k; ++i)
                mbar_wait(&bar.a_full[i % C::kStagesK], (uint32_t)(i / C::kStagesK) & 1u, abortp);
            for (int i = issued_v > C::kStages ? issued_v - C::kStages : 0; i < issued_v; ++i)
                mbar_wait(&bar.b_full[i % C::kStages], (uint32_t)(i / C::kStages) & 1u, abortp);
        }
    } else if (warp == kMmaWarp) {
        if (E > 0) {   // every lane runs the issue loop (converged); elect.sync inside the wrappers picks the issuing lane
            bool ok = mbar_wait_warp(&bar.fixed_full, 0, abortp);
            tc_fence_after();
            // low descriptor words of the operands (see make_desc): K-major views for S and dP, MN-major view of K for dQ
            const uint32_t q_lo = desc_lo_kmajor(smem_u32(sQ)), g_lo = desc_lo_kmajor(smem_u32(sdO));
            const uint32_t k_lo = desc_lo_kmajor(smem_u32(sK)), v_lo = desc_lo_kmajor(smem_u32(sV));
            const uint32_t kt_lo = desc_lo_mnmajor(smem_u32(sK), kPanel);
            auto issue_s = [&](int e) -> bool {             // S(e) = Q K(e)^T into the ping/pong buffer e & 1
                const int s = e % C::kStagesK;
                if (!mbar_wait_warp(&bar.a_full[s], (uint32_t)(e / C::kStagesK) & 1u, abortp)) return false;
                tc_fence_after();
                const uint32_t ka = k_lo + s * (C::kTile >> 4);
#pragma unroll
                for (int k = 0; k < DH / 16; ++k)
                    mma_ss_elect(tmem + kColS + (e & 1) * 128, make_desc(q_lo + kstep_off(k, kPanel)), make_desc(ka + kstep_off(k, kPanel)),
                           C::kIdescS, k > 0);
                mma_commit_elect(&bar.s_full[e & 1]);
                return true;
            };
            if (ok) ok = issue_s(0);
            for (int e = 0; e < E && ok; ++e) {
                const int s = e % C::kStagesK, sv = e % C::kStages;
                if (!mbar_wait_warp(&bar.b_full[sv], (uint32_t)(e / C::kStages) & 1u, abortp)) { ok = false; break; }
                tc_fence_after();
                const uint32_t va = v_lo + sv * (C::kTile >> 4), kta = kt_lo + s * (C::kTile >> 4);
#pragma unroll
                for (int k = 0; k < DH / 16; ++k)          // dP(e) = dO V(e)^T  (dS(e-1), which shares the columns, was consumed by dQ(e-1) issued before)
                    mma_ss_elect(tmem + kColDP, make_desc(g_lo + kstep_off(k, kPanel)), make_desc(va + kstep_off(k, kPanel)), C::kIdescS, k > 0);
                mma_commit_elect(&bar.dp_full);
                mma_commit_elect(&bar.b_empty[sv]);
                if (e + 1 < E && !issue_s(e + 1)) { ok = false; break; }
                // dQ += dS(e) K(e), in the two parts in which the element-wise threads hand dS over (32 of each thread's
                // 64 columns: K-steps {0, 1, 4, 5}, then {2, 3, 6, 7}), so that the first half runs under the second
#pragma unroll
                for (int part = 0; part < 2; ++part) {
                    if (!mbar_wait_warp(&bar.ds_part[part], (uint32_t)e & 1u, abortp)) { ok = false; break; }
                    tc_fence_after();
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int k = (i >> 1) * 4 + part * 2 + (i & 1);
                        mma_ts_elect(tmem + kColAcc, tmem + kColDP + packed_half_col(k), make_desc(kta + k * (2048 >> 4)), C::kIdescAcc,
                               (e > 0 || part > 0 || i > 0) ? 1u : 0u);
                    }
                }
                if (!ok) break;
                mma_commit_elect(&bar.a_empty[s]);
            }
            if (ok) mma_commit_elect(&bar.acc_done);
        }
    } else {
        // ------------------------------------------------------------ element-wise warpgroups (thread = query row, 64 of the 128 columns)
        const int w = warp >> 2;
        const int r = tid & 127;
        const long long t = m0 + r;
        const bool row_valid = t < p.T;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t dp_addr = tmem + lane_base + kColDP + w * 64;
        float Dt = 0.f, bias[3] = {-INFINITY, -INFINITY, -INFINITY};
        if (row_valid) {
            Dt = p.statD[bh * p.Tpad + t];
#pragma unroll
            for (int l = 0; l < 3; ++l) {
                bias[l] = p.statB[l][bh * p.Tpad + t];
            }
        }
        float Al[3] = {0.f, 0.f, 0.f}, Sl[3] = {0.f, 0.f, 0.f};   // per level: sum p dP and sum p over this thread's columns
        bool ok = true;
        int e = 0;
#pragma unroll
        for (int l = 0; l < 3; ++l) {
            if (!ok || first[l] == end[l]) continue;
            long long lo = 0, hi = 0;
            if (row_valid) visible_range(l, t + p.q_offset, p.window, p.n[l], 0, lo, hi);
            int full_first = 0, full_end = 0;
            {
                long long lo_f, hi_f, lo_l, hi_l;
                visible_range(l, m0 + p.q_offset, p.window, p.n[l], 0, lo_f, hi_f);
                visible_range(l, m_last + p.q_offset, p.window, p.n[l], 0, lo_l, hi_l);
                full_first = (int)((lo_l + kBlk - 1) / kBlk);
                full_end = (int)(hi_f / kBlk);
                if (m_last - m0 + 1 < kBlk) full_end = full_first;          // ragged query tile: always mask
            }
            // sums over this thread's columns as packed pairs (even, odd column)
            uint64_t a2 = pack2(0.f, 0.f), z2 = a2;
            const float bl = bias[l];
            const uint64_t scale2 = pack2(p.scale_log2, p.scale_log2), bl2 = pack2(bl, bl), negD2 = pack2(-Dt, -Dt);
            for (int kt = first[l]; kt < end[l]; ++kt, ++e) {
                // phase 1: p = 2^(s * scale + bias) for this thread's 64 columns (needs S only)
                ok = mbar_wait(&bar.s_full[e & 1], (uint32_t)(e >> 1) & 1u, abortp);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                float pr[64];
                {
                    const uint32_t s_addr = tmem + lane_base + kColS + (e & 1) * 128 + w * 64;
                    tmem_ld32(s_addr, reinterpret_cast<uint32_t*>(pr));
                    tmem_ld32(s_addr + 32, reinterpret_cast<uint32_t*>(pr) + 32);
                    tmem_ld_wait();
                }
                if (!(kt >= full_first && kt < full_end)) {
                    const long long j0 = (long long)kt * kBlk + w * 64;
                    const int c_lo = (int)max(-1LL, min(lo - j0, 64LL));
                    const int c_hi = (int)max(-1LL, min(hi - j0, 64LL));
#pragma unroll
                    for (int c = 0; c < 64; ++c)
                        if (c < c_lo || c >= c_hi) pr[c] = -INFINITY;
                }
#pragma unroll
                for (int c = 0; c < 64; c += 2) {
                    float x0, x1;
                    unpack2(fma2(pack2(pr[c], pr[c + 1]), scale2, bl2), x0, x1);
                    pr[c] = ex2(x0);
                    pr[c + 1] = ex2(x1);
                    z2 = add2(z2, pack2(pr[c], pr[c + 1]));
                }
                // phase 2: dS = p (dP - D), written (bf16) over the dP columns just read
                ok = mbar_wait(&bar.dp_full, (uint32_t)e & 1u, abortp);
                ok = __all_sync(0xffffffffu, ok);
                if (!ok) break;
                tc_fence_after();
                float dp[64];
                tmem_ld32(dp_addr, reinterpret_cast<uint32_t*>(dp));
                tmem_ld32(dp_addr + 32, reinterpret_cast<uint32_t*>(dp) + 32);
                tmem_ld_wait();
                uint32_t pk[16];
                auto ds_cols = [&](int c_from, int c_to, int c_base) {
#pragma unroll
                    for (int c = c_from; c < c_to; c += 2) {
                        const uint64_t p2 = pack2(pr[c], pr[c + 1]), d2 = pack2(dp[c], dp[c + 1]);
                        a2 = fma2(p2, d2, a2);
                        float s0, s1;
                        unpack2(mul2(p2, add2(d2, negD2)), s0, s1);
                        pk[(c - c_base) / 2] = pack_bf16(s0, s1);
                    }
                };
                auto hand_over = [&](int part) {
                    tmem_st_wait();
                    tc_fence_before();
                    __syncwarp();
                    if (lane == 0) mbar_arrive(&bar.ds_part[part]);
                };
                ds_cols(0, 32, 0);
                tmem_st16(dp_addr, pk);
                ds_cols(32, 48, 32);
                hand_over(0);                                // the first part's store has completed by now
                ds_cols(48, 64, 32);
                tmem_st16(dp_addr + 16, pk);
                hand_over(1);
            }
            {
                float a0, a1, z0, z1;
                unpack2(a2, a0, a1);
                unpack2(z2, z0, z1);
                Al[l] = a0 + a1;
                Sl[l] = z0 + z1;
            }
        }
        // ------------------------------------------------------------ epilogue
        if (ok && E > 0) {
            ok = mbar_wait(&bar.acc_done, 0, abortp);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            tc_fence_after();
            __nv_bfloat16* out = p.dQ + (bh * p.T + t) * DH;
#pragma unroll
            for (int c0 = w * (DH / 2); c0 < (w + 1) * (DH / 2); c0 += 32) {
                uint32_t o[32];
                if (E > 0) {
                    tmem_ld32(tmem + lane_base + kColAcc + c0, o);
                    tmem_ld_wait();
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = 0u;
                }
                if (row_valid) store_row_bf16(out + c0, o, p.scale);
            }
        }
        // Gate-logit gradient of this head: G_l = sum_{j in l} p (dP - D').  D' = sum p dP / sum p equals
        // dO . O in exact arithmetic but does not inherit the rounding of O to bf16, so sum_l G_l = 0 holds
        // to fp32 accuracy.  The two warpgroups hold disjoint columns: add their partial sums first.
        if (w == 1) {
#pragma unroll
            for (int l = 0; l < 3; ++l) { gsm[r][l] = Al[l]; gsm[r][3 + l] = Sl[l]; }
        }
        softmax_group_sync();
        if (w == 0 && ok && row_valid) {
            float a[3], z[3];
#pragma unroll
            for (int l = 0; l < 3; ++l) { a[l] = Al[l] + gsm[r][l]; z[l] = Sl[l] + gsm[r][3 + l]; }
            const float ztot = z[0] + z[1] + z[2];
            const float dd = ztot > 0.f ? (a[0] + a[1] + a[2]) / ztot : 0.f;
            float* g = p.Gpart + (bh * p.T + t) * 3;
#pragma unroll
            for (int l = 0; l < 3; ++l) g[l] = a[l] - z[l] * dd;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (tid == 0 && wait_ctl.abort) atomicExch(p.status, (unsigned int)MKA_ERR_TIMEOUT);
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
}

// ------------------------------------------------------------------------------------------ dK, dV
template <int DH>
__global__ void __launch_bounds__(kThreads, 1) bwd_dkv_tc_kernel(const __grid_constant__ BwdMaps maps, const BwdTcParams p) {
    using C = BCfg<DH>;
    constexpr uint32_t kColS = 0, kColDP = 128, kColDK = 256, kColDV = 256 + DH;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* sK = smem;
    uint8_t* sV = sK + C::kTile;
    uint8_t* sQ = sV + C::kTile;                          // kStages tiles
    uint8_t* sdO = sQ + C::kStages * C::kTile;            // kStages tiles
    // Operand slabs of the extra K-step (16 columns, no swizzle: 8-row x 16-byte core matrices, the two of a row group
    // 128 bytes apart, row groups 256 bytes apart).  sAugQ: per stage, [query][k] = the query's exponent bias divided by
    // the score scale, split into three bf16 terms (k = 0..2), then [query][k] = -D_t split the same way; sAugK: ones in
    // k = 0..2 for every key.  S^T + bias / scale and dP^T - D then come out of the tensor pipe, and the element-wise
    // threads need no per-column operand at all.
    uint8_t* sAugQ = sdO + C::kStages * C::kTile;          // kStages x {bias slab, D slab}
    uint8_t* sAugK = sAugQ + C::kStages * 2 * C::kAugBytes;
    __shared__ BwdBarriers bar;
    __shared__ uint32_t tmem_base_slot;
    __shared__ WaitCtl wait_ctl;

    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);   // tid >> 5, but provably warp-uniform for the compiler
    const int b = blockIdx.z, h = blockIdx.y;               // h: KV head; its query heads are h * G .. h * G + G - 1
    // key tiles in decreasing order of work: L3 (seen by every query), L2 from the oldest key on, L1
    int lvl, kt;
    {
        int x = blockIdx.x;
        if (x < p.kv_tiles[2]) { lvl = 2; kt = x; }
        else if (x < p.kv_tiles[2] + p.kv_tiles[1]) { lvl = 1; kt = x - p.kv_tiles[2]; }
        else { lvl = 0; kt = x - p.kv_tiles[2] - p.kv_tiles[1]; }
    }
    const long long n = p.n[lvl];
    const long long j0 = (long long)kt * kBlk;
    const long long j_last = (j0 + kBlk - 1 < n - 1) ? j0 + kBlk - 1 : n - 1;
    // queries t (position t + q_offset) that can see a key of this tile
    long long t_lo = 0, t_hi = p.T;
    if (lvl == 0) { t_lo = j0 - p.q_offset; t_hi = j_last + p.window - p.q_offset; }
    else if (lvl == 1) { t_lo = j0 - p.q_offset; }
    if (t_lo < 0) t_lo = 0;
    if (t_hi > p.T) t_hi = p.T;
    const int first = t_hi > t_lo ? (int)(t_lo / kBlk) : 0;
    const int Eq = t_hi > t_lo ? (int)((t_hi + kBlk - 1) / kBlk) - first : 0;    // query tiles of ONE head that see this key tile
    const int E = Eq * p.kv_group;                          // the stream: head by head, each head's tiles in order

    // The thread that issues the copies sets the barriers up itself and requests the CTA's own K and V tiles at once,
    // before the CTA-wide start-up (slabs, TMEM allocation) that the copies' latency can run under.
    if (warp == kProducerWarp && lane == 0) {
        wait_ctl.abort = 0;
        wait_ctl.limit_ns = p.wait_limit_ns;
        mbar_init(&bar.fixed_full, 1);
        for (int s = 0; s < kMaxStages; ++s) {               // full: the copy's bytes and the slab
            mbar_init(&bar.a_full[s], 2); mbar_init(&bar.a_empty[s], 1);
            mbar_init(&bar.b_full[s], 2); mbar_init(&bar.b_empty[s], 1);
        }
        mbar_init(&bar.s_full[0], 1);
        mbar_init(&bar.dp_full, 1);
        for (int i = 0; i < 2; ++i) { mbar_init(&bar.p_part[i], 8); mbar_init(&bar.ds_part[i], 8); }   // 8 = one arrival per element-wise warp
        mbar_init(&bar.acc_done, 1);
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
        if (E > 0) {
            mbar_expect_tx(&bar.fixed_full, 2 * C::kTile);
#pragma unroll
            for (int pn = 0; pn < C::kPanels; ++pn) {
                tma_load_4d(sK + pn * kPanel, &maps.k[lvl], pn * 64, (int)j0, h, b, &bar.fixed_full);
                tma_load_4d(sV + pn * kPanel, &maps.v[lvl], pn * 64, (int)j0, h, b, &bar.fixed_full);
            }
        }
    }
    // every slab zero (columns 3..15 stay zero), ones for the keys: all threads share the 36 KB
    for (int i = tid; i < (int)((C::kStages * 2 + 1) * C::kAugBytes / 16); i += kThreads)
        reinterpret_cast<uint4*>(sAugQ)[i] = make_uint4(0u, 0u, 0u, 0u);
    __syncthreads();
    if (tid < kBlk) *reinterpret_cast<uint4*>(sAugK + (tid & 7) * 16 + (tid >> 3) * 256) = make_uint4(0x3f803f80u, 0x00003f80u, 0u, 0u);
    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(512u) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_slot;
    volatile WaitCtl* abortp = &wait_ctl;

    if (warp == kProducerWarp) {
        if (E > 0) {   // the whole warp runs the loop (converged): lane 0 issues the copies, every lane writes its share of the slabs
            int issued = 0, issued_b = 0;
            const float inv_scale = 1.f / p.scale_log2;
            int hq = h * p.kv_group, eq = 0;                // query head and tile-within-head of stage e
            // this lane's four queries of a tile: their biases and D_t, fetched one tile ahead of the stage they go into
            auto fetch = [&](float4& bq, float4& dq) {
                const long long at = ((long long)b * p.H + hq) * p.Tpad + (long long)(first + eq) * kBlk + 4 * lane;
                bq = *reinterpret_cast<const float4*>(p.statB[lvl] + at);
                dq = *reinterpret_cast<const float4*>(p.statD + at);
            };
            float4 bq, dq;
            fetch(bq, dq);
            // Two rings: a stage's dO tile is free again after dV of its tile, its Q tile only after dK, one product later;
            // and the next tile's Q is what the issuing warp waits for first.  Each is re-filled as soon as it is free.
            for (int e = 0; e < E; ++e) {
                const int s = e % C::kStages;
                const uint32_t ph = (uint32_t)(e / C::kStages) & 1u;
                if (p.test_stall && e == E - 1) break;                 // test hook: the last tile never arrives
                const int tt = (first + eq) * kBlk;
                const float bv[4] = {bq.x, bq.y, bq.z, bq.w}, dv[4] = {dq.x, dq.y, dq.z, dq.w};
                if (!mbar_wait_warp(&bar.b_empty[s], ph ^ 1u, abortp)) break;
                if (lane == 0) {
                    mbar_expect_tx(&bar.b_full[s], C::kTile);
#pragma unroll
                    for (int pn = 0; pn < C::kPanels; ++pn)
                        tma_load_4d(sdO + s * C::kTile + pn * kPanel, &maps.dO, pn * 64, tt, hq, b, &bar.b_full[s]);
                }
                ++issued_b;
#pragma unroll
                for (int i = 0; i < 4; ++i) {                          // -D as three bf16 terms
                    const int r = 4 * lane + i;
                    *reinterpret_cast<uint4*>(sAugQ + (s * 2 + 1) * C::kAugBytes + (r & 7) * 16 + (r >> 3) * 256) = split3_bf16(-dv[i]);
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(&bar.b_full[s]);
                if (!mbar_wait_warp(&bar.a_empty[s], ph ^ 1u, abortp)) break;
                if (lane == 0) {
                    mbar_expect_tx(&bar.a_full[s], C::kTile);
#pragma unroll
                    for (int pn = 0; pn < C::kPanels; ++pn)
                        tma_load_4d(sQ + s * C::kTile + pn * kPanel, &maps.q, pn * 64, tt, hq, b, &bar.a_full[s]);
                }
                ++issued;
#pragma unroll
                for (int i = 0; i < 4; ++i) {                          // bias / scale as three bf16 terms
                    const int r = 4 * lane + i;
                    *reinterpret_cast<uint4*>(sAugQ + (s * 2) * C::kAugBytes + (r & 7) * 16 + (r >> 3) * 256) = split3_bf16(bv[i] * inv_scale);
                }
                asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                __syncwarp();
                if (lane == 0) mbar_arrive(&bar.a_full[s]);
                if (++eq == Eq) { eq = 0; ++hq; }
                if (e + 1 < E) fetch(bq, dq);
            }
            mbar_wait_warp(&bar.fixed_full, 0, abortp);
            for (int i = issued > C::kStages ? issued - C::kStages : 0; i < issued; ++i)
                mbar_wait_warp(&bar.a_full[i % C::kStages], (uint32_t)(i / C::kStages) & 1u, abortp);
            for (int i = issued_b > C::kStages ? issued_b - C::kStages : 0; i < issued_b; ++i)
                mbar_wait_warp(&bar.b_full[i % C::kStages], (uint32_t)(i / C::kStages) & 1u, abortp);
        }
    } else if (warp == kMmaWarp) {
        if (E > 0) {   // every lane runs the issue loop (converged); elect.sync inside the wrappers picks the issuing lane
            bool ok = mbar_wait_warp(&bar.fixed_full, 0, abortp);
            tc_fence_after();
            // low descriptor words (see make_desc): K-major views for S^T and dP^T, MN-major views of Q and dO for dK and dV
            const uint32_t k_lo = desc_lo_kmajor(smem_u32(sK)), v_lo = desc_lo_kmajor(smem_u32(sV));
            const uint32_t q_lo = desc_lo_kmajor(smem_u32(sQ)), g_lo = desc_lo_kmajor(smem_u32(sdO));
            const uint32_t qt_lo = desc_lo_mnmajor(smem_u32(sQ), kPanel), gt_lo = desc_lo_mnmajor(smem_u32(sdO), kPanel);
            const uint32_t augk_lo = desc_lo_flat(smem_u32(sAugK)), augq_lo = desc_lo_flat(smem_u32(sAugQ));
            auto issue_s = [&](int e) {                     // S^T(e) = K Q(e)^T   (P^T(e-1), which shares the columns, was consumed by dV(e-1) issued before; Q(e) has landed)
                const int s = e % C::kStages;
                tc_fence_after();
                const uint32_t qa = q_lo + s * (C::kTile >> 4);
#pragma unroll
                for (int k = 0; k < DH / 16; ++k)
                    mma_ss_elect(tmem + kColS, make_desc(k_lo + kstep_off(k, kPanel)), make_desc(qa + kstep_off(k, kPanel)), C::kIdescS, k > 0);
                mma_ss_elect(tmem + kColS, make_desc_flat(augk_lo), make_desc_flat(augq_lo + s * (2 * C::kAugBytes >> 4)), C::kIdescS, 1u);   // + bias_t / scale
                mma_commit_elect(&bar.s_full[0]);
            };
            auto issue_dp = [&](int e) -> bool {            // dP^T(e) = V dO(e)^T
                if (!mbar_wait_warp(&bar.b_full[e % C::kStages], (uint32_t)(e / C::kStages) & 1u, abortp)) return false;
                tc_fence_after();
                const uint32_t ga = g_lo + (e % C::kStages) * (C::kTile >> 4);
#pragma unroll
                for (int k = 0; k < DH / 16; ++k)
                    mma_ss_elect(tmem + kColDP, make_desc(v_lo + kstep_off(k, kPanel)), make_desc(ga + kstep_off(k, kPanel)), C::kIdescS, k > 0);
                mma_ss_elect(tmem + kColDP, make_desc_flat(augk_lo), make_desc_flat(augq_lo + ((e % C::kStages) * 2 + 1) * (C::kAugBytes >> 4)), C::kIdescS, 1u);   // - D_t
                mma_commit_elect(&bar.dp_full);
                return true;
            };
            if (ok) ok = mbar_wait_warp(&bar.a_full[0], 0, abortp);
            if (ok) issue_s(0);
            if (ok) ok = issue_dp(0);
            for (int e = 0; e < E && ok; ++e) {
                const int s = e % C::kStages;
                const uint32_t qta = qt_lo + s * (C::kTile >> 4), gta = gt_lo + s * (C::kTile >> 4);
                // dV += P^T(e) dO(e) and dK += dS^T(e) Q(e), each in the two parts in which the element-wise threads
                // hand their 64 columns over (K-steps {0, 1, 4, 5}, then {2, 3, 6, 7})
#pragma unroll
                for (int part = 0; part < 2; ++part) {
                    if (!mbar_wait_warp(&bar.p_part[part], (uint32_t)e & 1u, abortp)) { ok = false; break; }
                    tc_fence_after();
#pragma unroll
                    for (int i = 0; i < 4; ++i) {
                        const int k = (i >> 1) * 4 + part * 2 + (i & 1);
                        mma_ts_elect(tmem + kColDV, tmem + kColS + packed_half_col(k), make_desc(gta + k * (2048 >> 4)), C::kIdescAcc,
                               (e > 0 || part > 0 || i > 0) ? 1u : 0u);
                    }
                }
                if (!ok) break;
                mma_commit_elect(&bar.b_empty[s]);                     // dO(e) has had its last reader
                // S^T(e+1) needs Q(e+1), which can only be requested once dK(e-1) has released its stage; dK(e) needs dS^T(e)
                // from the element-wise threads.  Either may be ready first, and neither may wait for the other (a late
                // dK delays the release, the release the copy, the copy the next S^T): poll both.
                {
                    const int sn = (e + 1) % C::kStages;
                    const uint32_t phn = (uint32_t)((e + 1) / C::kStages) & 1u;
                    bool s_out = e + 1 >= E;
                    int dk_part = 0;
                    const unsigned long long t0 = gtimer();
                    while (!s_out || dk_part < 2) {
                        bool moved = false;
                        if (!s_out && __all_sync(0xffffffffu, mbar_try(&bar.a_full[sn], phn))) {
                            issue_s(e + 1);
                            s_out = moved = true;
                        }
                        if (dk_part < 2 && __all_sync(0xffffffffu, mbar_try(&bar.ds_part[dk_part], (uint32_t)e & 1u))) {
                            tc_fence_after();
#pragma unroll
                            for (int i = 0; i < 4; ++i) {
                                const int k = (i >> 1) * 4 + dk_part * 2 + (i & 1);
                                mma_ts_elect(tmem + kColDK, tmem + kColDP + packed_half_col(k), make_desc(qta + k * (2048 >> 4)), C::kIdescAcc,
                                       (e > 0 || dk_part > 0 || i > 0) ? 1u : 0u);
                            }
                            ++dk_part;
                            moved = true;
                        }
                        if (!moved) {                            // bounded like every other wait of the kernel
                            bool give_up = abortp->abort != 0;
                            if (!give_up && gtimer() - t0 > abortp->limit_ns) { abortp->abort = 1; give_up = true; }
                            if (__any_sync(0xffffffffu, give_up)) { ok = false; break; }
                        }
                    }
                }
                if (!ok) break;
                mma_commit_elect(&bar.a_empty[s]);
                if (e + 1 < E && !issue_dp(e + 1)) { ok = false; break; }
            }
            if (ok) mma_commit_elect(&bar.acc_done);
        }
    } else {
        // ------------------------------------------------------------ element-wise warpgroups (thread = key row, 64 of the 128 query columns)
        const int w = warp >> 2;
        const int r = tid & 127;
        const long long j = j0 + r;
        const bool row_valid = j < n;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t s_addr = tmem + lane_base + kColS + w * 64;
        const uint32_t dp_addr = tmem + lane_base + kColDP + w * 64;
        // queries [q_lo, q_hi) that see key j (the bound t < T is carried by the padded biases)
        long long q_lo = 0, q_hi = 0;
        if (row_valid) {
            q_lo = lvl == 2 ? 0 : j - p.q_offset;
            q_hi = lvl == 0 ? j + p.window - p.q_offset : (long long)p.Tpad;
        }
        const bool rows_full = j0 + kBlk - 1 < n;
        bool ok = true;
        int eq = 0;                                                    // tile within the current query head
        for (int e = 0; e < E; ++e) {
            const int s = e % C::kStages;
            const long long tt = (long long)(first + eq) * kBlk;       // first query of the tile
            if (++eq == Eq) eq = 0;
            // phase 1: P^T = 2^(scale * (s + bias_t / scale)) for this thread's 64 query columns; the sum comes from the tensor pipe
            ok = mbar_wait(&bar.s_full[0], (uint32_t)e & 1u, abortp);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            float pr[64];
            tmem_ld32(s_addr, reinterpret_cast<uint32_t*>(pr));
            tmem_ld32(s_addr + 32, reinterpret_cast<uint32_t*>(pr) + 32);
            tmem_ld_wait();
            // tiles whose every (key, query) pair is visible need no mask
            bool full = rows_full;
            if (lvl != 2) full = full && (j_last - p.q_offset <= tt);
            if (lvl == 0) full = full && (j0 + p.window - p.q_offset >= tt + kBlk);
            if (!full) {
                const long long c0 = tt + w * 64;
                const int c_lo = (int)max(-1LL, min(q_lo - c0, 64LL));
                const int c_hi = (int)max(-1LL, min(q_hi - c0, 64LL));
#pragma unroll
                for (int c = 0; c < 64; ++c)
                    if (c < c_lo || c >= c_hi) pr[c] = -INFINITY;
            }
            uint32_t pk[32];        // P^T rounded to bf16; phase 2 uses these same rounded values
            const uint64_t scale2 = pack2(p.scale_log2, p.scale_log2);
            auto p_cols = [&](int c_from, int c_to) {
#pragma unroll
                for (int c = c_from; c < c_to; c += 2) {
                    float x0, x1;
                    unpack2(mul2(pack2(pr[c], pr[c + 1]), scale2), x0, x1);
                    // Every other pair on the FMA pipe: the hand-over of P^T, not these threads' total work, is what the
                    // next score product waits for, and the special-function unit alone is the slower way there.
                    float p0, p1;
                    if ((c >> 1) & 1) { p0 = ex2(x0); p1 = ex2(x1); }
                    else exp2_pair_fma(x0, x1, p0, p1);
                    pk[c / 2] = pack_bf16(p0, p1);
                }
            };
            auto hand_over = [&](uint64_t* bar_part) {       // everything stored so far is in TMEM
                tmem_st_wait();
                tc_fence_before();
                __syncwarp();
                if (lane == 0) mbar_arrive(bar_part);
            };
            // each half of the thread's 64 columns goes out as soon as it is ready; the first half is handed over in
            // the middle of the second half's exponentials, when its store has long completed
            p_cols(0, 32);
            tmem_st16(s_addr, pk);
            p_cols(32, 48);
            hand_over(&bar.p_part[0]);
            p_cols(48, 64);
            tmem_st16(s_addr + 16, pk + 16);
            hand_over(&bar.p_part[1]);
            // phase 2: dS^T = P^T (dP^T - D_t), written over the columns just read; the difference comes from the tensor pipe
            ok = mbar_wait(&bar.dp_full, (uint32_t)e & 1u, abortp);
            ok = __all_sync(0xffffffffu, ok);
            if (!ok) break;
            tc_fence_after();
            tmem_ld32(dp_addr, reinterpret_cast<uint32_t*>(pr));
            tmem_ld32(dp_addr + 32, reinterpret_cast<uint32_t*>(pr) + 32);
            tmem_ld_wait();
            auto ds_cols = [&](int c_from, int c_to) {
#pragma unroll
                for (int c = c_from; c < c_to; c += 2) {
                    const float p0 = __uint_as_float(pk[c / 2] << 16), p1 = __uint_as_float(pk[c / 2] & 0xffff0000u);
                    float s0, s1;
                    unpack2(mul2(pack2(p0, p1), pack2(pr[c], pr[c + 1])), s0, s1);   // p (dP - D)
                    pk[c / 2] = pack_bf16(s0, s1);
                }
            };
            ds_cols(0, 32);
            tmem_st16(dp_addr, pk);
            ds_cols(32, 48);
            hand_over(&bar.ds_part[0]);
            ds_cols(48, 64);
            tmem_st16(dp_addr + 16, pk + 16);
            hand_over(&bar.ds_part[1]);
        }
        // ------------------------------------------------------------ epilogue: warpgroup 0 writes dK, 1 writes dV
        if (ok && E > 0) {
            ok = mbar_wait(&bar.acc_done, 0, abortp);
            ok = __all_sync(0xffffffffu, ok);
        }
        if (ok) {
            tc_fence_after();
            const LevelGradDev dL = p.dL[lvl];
            __nv_bfloat16* out = static_cast<__nv_bfloat16*>(w == 0 ? dL.dk : dL.dv) + b * dL.sb + h * dL.sh + j * dL.sn;
            const float mul = w == 0 ? p.scale : 1.f;
#pragma unroll
            for (int c0 = 0; c0 < DH; c0 += 32) {
                uint32_t o[32];
                if (E > 0) {
                    tmem_ld32(tmem + lane_base + (w == 0 ? kColDK : kColDV) + c0, o);
                    tmem_ld_wait();
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = 0u;
                }
                if (row_valid) store_row_bf16(out + c0, o, mul);
            }
        }
    }

    tc_fence_before();
    __syncthreads();
    if (tid == 0 && wait_ctl.abort) atomicExch(p.status, (unsigned int)MKA_ERR_TIMEOUT);
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(512u) : "memory");
}

template <int DH>
cudaError_t launch_t(const BwdParams& bp, unsigned int* status_word, cudaStream_t st) {
    using C = BCfg<DH>;
    const int Tpad = (bp.T + kBlk - 1) / kBlk * kBlk;
    const long long rows_pad = (long long)bp.B * bp.H * Tpad;
    float* statD = bp.stats;                              // the workspace holds D and the three bias arrays back to back
    float* statB[3];
    for (int l = 0; l < 3; ++l) statB[l] = bp.stats + (long long)(1 + l) * rows_pad;
    const long long sq_n = DH, sq_h = (long long)bp.T * DH, sq_b = (long long)bp.H * bp.T * DH;

    constexpr int kPrepRowsPerBlock = 8 * (32 / (DH / 8)) * 4;          // 8 warps x rows per pass x passes
    bwd_prep_kernel<DH><<<(unsigned)((rows_pad + kPrepRowsPerBlock - 1) / kPrepRowsPerBlock), 256, 0, st>>>(
        static_cast<const __nv_bfloat16*>(bp.O), static_cast<const __nv_bfloat16*>(bp.dO), bp.LSE, bp.gate, bp.H, bp.T, Tpad,
        rows_pad, statD, statB[0], statB[1], statB[2]);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;

    BwdTcParams p;
    p.dQ = static_cast<__nv_bfloat16*>(bp.dQ);
    p.statD = statD;
    p.Gpart = bp.Gpart;
    for (int l = 0; l < 3; ++l) {
        p.statB[l] = statB[l];
        p.dL[l] = bp.dL[l];
        p.n[l] = bp.L[l].n;
        p.kv_tiles[l] = (int)((bp.L[l].n + 127) / 128);
    }
    p.B = bp.B; p.H = bp.H; p.T = bp.T; p.Tpad = Tpad; p.kv_group = bp.kv_group > 0 ? bp.kv_group : 1;
    const int H_kv = bp.H / p.kv_group;
    p.window = bp.window; p.q_offset = bp.q_offset;
    p.scale = bp.scale; p.scale_log2 = bp.scale * kLog2e;
    p.status = status_word;
    p.wait_limit_ns = wait_limit_ns();
    p.test_stall = bp.test_stall;

    // both kernels move 128-row tiles (box = 64 columns x 128 rows)
    {
        BwdMaps m;
        if (!make_bf16_map(&m.q, bp.Q, DH, bp.T, bp.H, bp.B, sq_n, sq_h, sq_b, 128) ||
            !make_bf16_map(&m.dO, bp.dO, DH, bp.T, bp.H, bp.B, sq_n, sq_h, sq_b, 128))
            return cudaErrorNotSupported;
        for (int l = 0; l < 3; ++l) {
            if (bp.L[l].n == 0) { m.k[l] = m.q; m.v[l] = m.q; continue; }
            if (!make_bf16_map(&m.k[l], bp.L[l].k, DH, bp.L[l].n, H_kv, bp.B, bp.L[l].sn, bp.L[l].sh, bp.L[l].sb, kBlk) ||
                !make_bf16_map(&m.v[l], bp.L[l].v, DH, bp.L[l].n, H_kv, bp.B, bp.L[l].sn, bp.L[l].sh, bp.L[l].sb, kBlk))
                return cudaErrorNotSupported;
        }
        e = cudaFuncSetAttribute(bwd_dq_tc_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::kSmemDq);
        if (e != cudaSuccess) return e;
        dim3 grid((bp.T + 127) / 128, bp.H, bp.B);
        bwd_dq_tc_kernel<DH><<<grid, kThreads, C::kSmemDq, st>>>(m, p);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    const int tiles = p.kv_tiles[0] + p.kv_tiles[1] + p.kv_tiles[2];
    if (tiles > 0) {
        BwdMaps m;
        if (!make_bf16_map(&m.q, bp.Q, DH, bp.T, bp.H, bp.B, sq_n, sq_h, sq_b, kBlk) ||
            !make_bf16_map(&m.dO, bp.dO, DH, bp.T, bp.H, bp.B, sq_n, sq_h, sq_b, kBlk))
            return cudaErrorNotSupported;
        for (int l = 0; l < 3; ++l) {
            if (bp.L[l].n == 0) { m.k[l] = m.q; m.v[l] = m.q; continue; }
            if (!make_bf16_map(&m.k[l], bp.L[l].k, DH, bp.L[l].n, H_kv, bp.B, bp.L[l].sn, bp.L[l].sh, bp.L[l].sb, 128) ||
                !make_bf16_map(&m.v[l], bp.L[l].v, DH, bp.L[l].n, H_kv, bp.B, bp.L[l].sn, bp.L[l].sh, bp.L[l].sb, 128))
                return cudaErrorNotSupported;
        }
        e = cudaFuncSetAttribute(bwd_dkv_tc_kernel<DH>, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)C::kSmemDkv);
        if (e != cudaSuccess) return e;
        dim3 grid(tiles, H_kv, bp.B);
        bwd_dkv_tc_kernel<DH><<<grid, kThreads, C::kSmemDkv, st>>>(m, p);
        if ((e = cudaGetLastError()) != cudaSuccess) return e;
    }
    return launch_bwd_dgate(bp.Gpart, bp.B, bp.H, bp.T, bp.dG, st);
}

}  // namespace

bool bwd_tc_eligible(const BwdParams& p, int dtype) {
    if (dtype != MKA_BF16) return false;
    if (p.d != 64 && p.d != 128) return false;
    if (p.H > 65535 || p.B > 65535) return false;
    for (int l = 0; l < 3; ++l) {
        const LevelDev& L = p.L[l];
        if (L.n == 0) continue;
        if (L.n > 0x7fffffffLL - 256) return false;
        if (L.sn % 8 || L.sn <= 0) return false;
        if (p.H / (p.kv_group > 0 ? p.kv_group : 1) > 1 && (L.sh % 8 || L.sh <= 0)) return false;
        if (p.B > 1 && (L.sb % 8 || L.sb <= 0)) return false;
        if (p.dL[l].sn % 8 || p.dL[l].sh % 8 || p.dL[l].sb % 8) return false;
    }
    return tensor_map_encoder_available();
}

cudaError_t launch_bwd_tc(const BwdParams& p, unsigned int* status_word, cudaStream_t st) {
    if (p.B == 0 || p.H == 0 || p.T == 0) return cudaSuccess;
    return p.d == 128 ? launch_t<128>(p, status_word, st) : launch_t<64>(p, status_word, st);
}

}  // namespace mka
