// Tensor-core forward of Eq. 5 for bf16 on sm_100a: TMA -> shared memory -> tcgen05.mma -> TMEM.
//
// A CTA owns 128-row query tiles of one (batch, head) -- two of them ("ping" and "pong", 256 rows) at d = 128, one at
// d = 64, where two CTAs share an SM -- and walks ONE level-ordered list of 128-row key tiles: all visible L1 tiles,
// then L2, then L3.  A single running (max, sum) per row spans the three levels (the max shift of Eq. 11-14); the gate
// enters as a per-row, per-level additive bias log2(lambda) inside the exponent, so that
//     p = 2^(s * tau * log2(e) + log2(lambda_l) - m)  =  lambda_l * exp(s*tau - m')
// which is exactly the gated, un-normalised weight of Eq. 5.  One normalisation at the end.
//
// Warp roles (d = 128: 320 threads, d = 64: 384 threads):
//   softmax warps    thread = one query row (TMEM lane) x 128 key columns at d = 128 (four warps per query tile), x 64
//                    columns at d = 64 (eight warps: warp = (column half, lane quarter); the two threads of a row agree
//                    on the row maximum through shared memory and a 256-thread barrier).  Reads S from TMEM, applies
//                    bias and masks, running max, exp2, packs the weights to bf16 and writes them to TMEM in parts of
//                    32 keys (at d = 128 over the columns S occupied), rescales the O accumulator when the running
//                    maximum grows by more than 2^8 (lazy rescale), and does the epilogue.
//   next warp        producer: one lane issues the TMA loads of Q and of the K / V tile list into 128-byte-swizzled
//                    shared-memory rings (one mbarrier pair per stage); with paged levels the whole warp produces.
//   next warp        issues every tcgen05.mma (the warp runs its loop converged, one elected lane issues):
//                    S_q = Q_q K^T (both operands from shared memory) and O_q += P_q V (P from TMEM, V from shared
//                    memory, N-major) in pieces that follow the parts of P, so that most of the product runs under the
//                    remaining exponentials.  At d = 128 the order is  S0(e)  O1(e-1)  S1(e)  O0(e):  each tile's
//                    softmax overlaps the other tile's products.
//   d = 64 only      two idle warps complete the last warpgroup, so that registers can be moved from it to the softmax
//                    warpgroups (setmaxnreg): two CTAs per SM leave 80 registers per thread at launch.
// TMEM: S tiles first (128 columns each), then the O accumulators (d columns each); at d = 64 a P region of 64 columns
// per query tile follows, and S_q(e+1) is multiplied while the softmax of S_q(e) runs (the hand-off is "S is in
// registers", not "P has been consumed").  d = 128 uses all 512 columns, d = 64 256.
// What bounds the d = 128 kernel is the chain  softmax_q(e) -> O_q += P V -> S_q(e+1) -> softmax_q(e+1):  a key tile
// costs the tensor pipe 2048 cycles and the special-function unit 2048 cycles for the two query tiles, but S_q(e+1)
// cannot be written before P_q(e), which lies over S_q(e), has been consumed, and TMEM has no room for a second S.
// Every mbarrier wait is bounded by a wall-clock limit; on expiry the CTA raises a flag in shared
// memory, writes the device status word, lets every role drain, frees TMEM and returns.
#include "tc_ptx.cuh"

namespace mka {
namespace {

constexpr uint32_t kPanelBytes = 128 * 128;          // [128 rows][64 bf16] with 128-byte rows
constexpr float kRescaleThreshold = 8.0f;            // log2 units

struct TcMaps {
    CUtensorMap q;
    CUtensorMap k[3];
    CUtensorMap v[3];
};

struct TcParams {
    __nv_bfloat16* O;
    float* LSE;
    const float* gate;
    long long n[3];
    int B, H, T;
    int kv_group;            // query heads per KV head
    int window, q_offset;
    float scale_log2;
    unsigned int* status;
    unsigned long long wait_limit_ns;
    int test_stall;          // test hook (MKA_FLAG_TEST_STALL): the producer leaves out the last key tile of every CTA
    // paged levels: a 128-row key tile is assembled from boxes of box_rows rows, one page-table look-up per box
    int paged;
    const int* table[3];
    long long table_stride[3], table_head_stride[3];
    int page_shift[3], box_rows[3], pool_pages[3];
    const int* rows[3];      // per-sequence rows of a level (clamped to [0, n]), or null
    int deal;                // (batch, head) pairs per group of blocks dealt by query block (1 = pair by pair)
};

template <int DH>
struct Cfg {
    // d = 128: one CTA per SM with two query tiles (all 512 TMEM columns); a softmax thread owns a whole query row
    // (128 key columns, 168 registers per thread).
    // d = 64: the scores of one key tile cost the special-function unit as much as at d = 128 but only half the
    // tensor work, and the tile lists of the training shapes are short; there a CTA takes ONE query tile (256 TMEM
    // columns) and two CTAs share the SM, so that one CTA's start-up, waits and epilogue run under the other's steady
    // state.  Two CTAs leave 80 registers per thread, so a row is split between two threads (64 columns each), and
    // registers are moved from the last warpgroup to the softmax warpgroups.
    static constexpr int kNumQ = DH == 128 ? 2 : 1;
    static constexpr int kCtasPerSm = DH == 128 ? 1 : 2;
    static constexpr int kSplit = DH == 128 ? 1 : 2;           // threads per query row
    static constexpr int kCols = kTileN / kSplit;             // key columns of one softmax thread
    static constexpr int kParts = kCols / 32;                 // the weights of a tile are handed over in parts of 32 keys per thread
    static constexpr int kRowWarps = 4 * kSplit;              // softmax warps per query tile
    static constexpr int kSoftmaxWarps = kRowWarps * kNumQ;
    static constexpr bool kMoveRegs = kSplit == 2;            // re-divide the registers between the warpgroups (setmaxnreg)
    // with kMoveRegs the last warpgroup is completed by two idle warps: setmaxnreg is a warpgroup-wide instruction
    static constexpr int kThreads = (kSoftmaxWarps + (kMoveRegs ? 4 : 2)) * 32;
    static constexpr int kProducerWarp = kSoftmaxWarps, kMmaWarp = kSoftmaxWarps + 1;
    // What the warpgroups hold after the move must not exceed what the launch gave the CTA, or the increase would
    // wait forever:  384 threads x 80 registers at launch = 256 x 104 + 128 x 32.
    static constexpr int kRegsLaunch = 80, kRegsSoftmax = 104, kRegsOther = 32;
    static_assert(!kMoveRegs || kSoftmaxWarps * 32 * kRegsSoftmax + 4 * 32 * kRegsOther <= kThreads * kRegsLaunch, "register pool of the CTA exceeded");
    static_assert(!kMoveRegs || kThreads * kCtasPerSm * (kRegsLaunch + 8) > 65536, "the launch would get more than kRegsLaunch registers per thread");
    static constexpr int kPanels = DH / 64;
    static constexpr uint32_t kTileBytes = kPanels * kPanelBytes;
    static constexpr int kStages = 2;
    static constexpr uint32_t kSmemBytes = (kNumQ + 2 * kStages) * kTileBytes + 1024;
    static constexpr uint32_t kIdescQK = (1u << 4) | (1u << 7) | (1u << 10) | ((uint32_t)(kTileN >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
    // With d = 64 the O accumulator leaves TMEM columns free: P gets a region of its own there instead of
    // overwriting S, so S(e+1) can be multiplied while the softmax of S(e) is still running.
    static constexpr bool kSeparateP = DH == 64;
    static constexpr uint32_t kColO = kNumQ * kTileN;          // first accumulator column (S tiles come first)
    static constexpr uint32_t kColP = kColO + kNumQ * DH;     // first P column when kSeparateP
    static constexpr uint32_t kTmemCols = DH == 128 ? 512u : 256u;
    static_assert(kColP + (kSeparateP ? kNumQ * (kTileN / 2) : 0) <= kTmemCols, "TMEM columns exceeded");
    static constexpr uint32_t kIdescPV = (1u << 4) | (1u << 7) | (1u << 10) | (1u << 16) | ((uint32_t)(DH >> 3) << 17) | ((uint32_t)(kTileM >> 4) << 24);
};

constexpr int kMaxQ = 2;

struct Barriers {
    uint64_t q_full;
    uint64_t k_full[4], k_empty[4], v_full[4], v_empty[4];
    uint64_t s_full[kMaxQ], p_part[kMaxQ][4], pv_done[kMaxQ];   // p_part: the first / second 32 keys of both column halves are written
    uint64_t s_free[kMaxQ];   // d = 64 only: the warpgroup has read S(e) into registers, S(e+1) may overwrite it
};

// Key-tile range [first, end) of a block of query rows [r0, r1] (inclusive) on one level.
__device__ __forceinline__ void tile_range(int level, long long r0, long long r1, int q_offset, int window, long long n,
                                           int& first, int& end) {
    long long lo_f, hi_f, lo_l, hi_l;
    visible_range(level, r0 + q_offset, window, n, 0, lo_f, hi_f);
    visible_range(level, r1 + q_offset, window, n, 0, lo_l, hi_l);
    const long long hi = hi_l > hi_f ? hi_l : hi_f;
    if (hi <= lo_f) { first = end = 0; return; }
    first = (int)(lo_f / kTileN);
    end = (int)((hi + kTileN - 1) / kTileN);
}

template <int DH, bool kPaged>
__global__ void __launch_bounds__(Cfg<DH>::kThreads, Cfg<DH>::kCtasPerSm) fwd_tc_kernel(const __grid_constant__ TcMaps maps, const TcParams p) {
    using C = Cfg<DH>;
    extern __shared__ uint8_t smem_raw[];
    uint8_t* smem = reinterpret_cast<uint8_t*>((reinterpret_cast<uintptr_t>(smem_raw) + 1023) & ~static_cast<uintptr_t>(1023));
    uint8_t* sQ = smem;                                   // C::kNumQ tiles
    uint8_t* sK = sQ + C::kNumQ * C::kTileBytes;             // kStages tiles
    uint8_t* sV = sK + C::kStages * C::kTileBytes;        // kStages tiles
    __shared__ Barriers bar;
    __shared__ uint32_t tmem_base_slot;
    __shared__ WaitCtl wait_ctl;
    __shared__ float xmax[2][C::kNumQ][C::kSplit][kTileM];           // row maxima of the two column halves, double-buffered by tile parity
    __shared__ float lsum[C::kNumQ][C::kSplit][kTileM];              // row sums of the two column halves (epilogue)

    const int tid = threadIdx.x, lane = tid & 31;
    const int warp = __shfl_sync(0xffffffffu, tid >> 5, 0);   // tid >> 5, but provably warp-uniform for the compiler
    // Blocks start in the order of their linear index.  Within a group of p.deal (batch, head) pairs the blocks are
    // dealt by query block, heaviest (latest rows) first for every pair of the group, then the next lighter one: the
    // launch then ends with the group's lightest blocks instead of the last head's heaviest.
    const int lin = blockIdx.x + gridDim.x * (blockIdx.y + gridDim.y * blockIdx.z);      // fewer than 2^31 blocks
    const int per_group = p.deal * (int)gridDim.x;
    const int grp = lin / per_group, in_grp = lin - grp * per_group;
    const int pairs_here = min(p.deal, (int)(gridDim.y * gridDim.z) - grp * p.deal);
    const int hb = grp * p.deal + in_grp % pairs_here;
    const int b = hb / (int)gridDim.y, h = hb - b * (int)gridDim.y;
    const int qpair = gridDim.x - 1 - in_grp / pairs_here;
    const long long m0 = (long long)qpair * (C::kNumQ * kTileM);
    const long long m_last = (m0 + C::kNumQ * kTileM - 1 < p.T - 1) ? m0 + C::kNumQ * kTileM - 1 : p.T - 1;

    if (tid == 0) {
        wait_ctl.abort = 0;
        wait_ctl.limit_ns = p.wait_limit_ns;
        mbar_init(&bar.q_full, 1);
        for (int s = 0; s < 4; ++s) {
            mbar_init(&bar.k_full[s], 1); mbar_init(&bar.k_empty[s], 1);
            mbar_init(&bar.v_full[s], 1); mbar_init(&bar.v_empty[s], 1);
        }
        for (int q = 0; q < C::kNumQ; ++q) {
            mbar_init(&bar.s_full[q], 1); mbar_init(&bar.pv_done[q], 1);
            for (int i = 0; i < 4; ++i) mbar_init(&bar.p_part[q][i], C::kRowWarps);   // one arrival per softmax warp
            mbar_init(&bar.s_free[q], C::kRowWarps);
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == 0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;" ::"r"(smem_u32(&tmem_base_slot)), "r"(C::kTmemCols) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    tc_fence_before();
    __syncthreads();
    tc_fence_after();
    const uint32_t tmem = tmem_base_slot;
    volatile WaitCtl* abortp = &wait_ctl;

    // rows of the three levels for this sequence
    long long nl[3];
#pragma unroll
    for (int l = 0; l < 3; ++l) {
        nl[l] = p.n[l];
        if (kPaged && p.rows[l]) {
            const long long r = p.rows[l][b];
            nl[l] = r < 0 ? 0 : (r < p.n[l] ? r : p.n[l]);
        }
    }
    // the CTA's level-ordered key-tile list (same closed form in every role)
    int first[3], end[3];
#pragma unroll
    for (int l = 0; l < 3; ++l) {
        if (nl[l] > 0) tile_range(l, m0, m_last, p.q_offset, p.window, nl[l], first[l], end[l]);
        else first[l] = end[l] = 0;
    }
    const int E = (end[0] - first[0]) + (end[1] - first[1]) + (end[2] - first[2]);

    if (warp >= C::kSoftmaxWarps) {
    if constexpr (C::kMoveRegs) asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(C::kRegsOther));
    if (warp == C::kProducerWarp && kPaged) {
        // Paged levels: the whole warp produces.  Lane i owns box i of every key tile (a box = the rows of one page
        // that fall into the tile): it looks its page up while the warp waits for the stage to drain and issues its
        // own copies, so a tile costs one table round trip (overlapped) and four warp-wide copy instructions.
        if (lane == 0) {
            mbar_expect_tx(&bar.q_full, C::kNumQ * C::kTileBytes);
#pragma unroll
            for (int q = 0; q < C::kNumQ; ++q)
#pragma unroll
                for (int pn = 0; pn < C::kPanels; ++pn)
                    tma_load_4d(sQ + q * C::kTileBytes + pn * kPanelBytes, &maps.q, pn * 64, (int)(m0 + q * kTileM), h, b, &bar.q_full);
        }
        int issued = 0;
        bool ok = true;
        const int kvh = h / p.kv_group;
        for (int l = 0; l < 3 && ok; ++l) {
            if (first[l] >= end[l]) continue;
            const int* tab = p.table[l] + (long long)b * p.table_stride[l] + (long long)kvh * p.table_head_stride[l];
            const int rpb = p.box_rows[l];
            const bool mine = lane < kTileN / rpb;
            const int in_mask = (1 << p.page_shift[l]) - 1;
            for (int kt = first[l]; kt < end[l]; ++kt) {
                const int s = issued % C::kStages;
                const uint32_t ph = (uint32_t)(issued / C::kStages) & 1u;
                // a box past the level's last row is aimed past the pool, where the copy engine fills zeros as it does
                // past a dense level's end
                const long long row = (long long)kt * kTileN + lane * rpb;
                int page = p.pool_pages[l];
                if (mine && row < nl[l]) page = tab[row >> p.page_shift[l]];
                const int in_row = (int)(row & in_mask);
                if (!mbar_wait_warp(&bar.k_empty[s], ph ^ 1u, abortp)) { ok = false; break; }
                if (lane == 0) mbar_expect_tx(&bar.k_full[s], C::kTileBytes);
                __syncwarp();
                if (mine) {
#pragma unroll
                    for (int pn = 0; pn < C::kPanels; ++pn)
                        tma_load_4d(sK + s * C::kTileBytes + pn * kPanelBytes + lane * rpb * 128, &maps.k[l], pn * 64, in_row, kvh, page,
                                    &bar.k_full[s]);
                }
                if (!mbar_wait_warp(&bar.v_empty[s], ph ^ 1u, abortp)) {           // gave up with this stage's K copies in flight
                    mbar_wait_warp(&bar.k_full[s], ph, abortp);
                    ok = false;
                    break;
                }
                if (lane == 0) mbar_expect_tx(&bar.v_full[s], C::kTileBytes);
                __syncwarp();
                if (mine) {
#pragma unroll
                    for (int pn = 0; pn < C::kPanels; ++pn)
                        tma_load_4d(sV + s * C::kTileBytes + pn * kPanelBytes + lane * rpb * 128, &maps.v[l], pn * 64, in_row, kvh, page,
                                    &bar.v_full[s]);
                }
                ++issued;
            }
        }
        // Before leaving, make sure every copy issued has landed (bounded): the shared memory must not be handed to
        // another CTA with a bulk copy still in flight.  (A stage whose wait failed got no copies.)
        mbar_wait_warp(&bar.q_full, 0, abortp);
        for (int i = issued > C::kStages ? issued - C::kStages : 0; i < issued; ++i) {
            mbar_wait_warp(&bar.k_full[i % C::kStages], (uint32_t)(i / C::kStages) & 1u, abortp);
            mbar_wait_warp(&bar.v_full[i % C::kStages], (uint32_t)(i / C::kStages) & 1u, abortp);
        }
    } else if (warp == C::kProducerWarp) {
        if (lane == 0) {
            mbar_expect_tx(&bar.q_full, C::kNumQ * C::kTileBytes);
#pragma unroll
            for (int q = 0; q < C::kNumQ; ++q)
#pragma unroll
                for (int pn = 0; pn < C::kPanels; ++pn)
                    tma_load_4d(sQ + q * C::kTileBytes + pn * kPanelBytes, &maps.q, pn * 64, (int)(m0 + q * kTileM), h, b, &bar.q_full);
            int issued_k = 0, issued_v = 0;
            bool ok = true;
            const int kvh = h / p.kv_group;
            for (int l = 0; l < 3 && ok; ++l) {
                for (int kt = first[l]; kt < end[l]; ++kt) {
                    if (p.test_stall && issued_k == E - 1) break;      // test hook: the last tile never arrives
                    const int e = issued_k;
                    const int s = e % C::kStages;
                    const uint32_t ph = (uint32_t)(e / C::kStages) & 1u;
                    if (!mbar_wait(&bar.k_empty[s], ph ^ 1u, abortp)) { ok = false; break; }
                    mbar_expect_tx(&bar.k_full[s], C::kTileBytes);
#pragma unroll
                    for (int pn = 0; pn < C::kPanels; ++pn)
                        tma_load_4d(sK + s * C::kTileBytes + pn * kPanelBytes, &maps.k[l], pn * 64, kt * kTileN, kvh, b, &bar.k_full[s]);
                    ++issued_k;
                    if (!mbar_wait(&bar.v_empty[s], ph ^ 1u, abortp)) { ok = false; break; }
                    mbar_expect_tx(&bar.v_full[s], C::kTileBytes);
#pragma unroll
                    for (int pn = 0; pn < C::kPanels; ++pn)
                        tma_load_4d(sV + s * C::kTileBytes + pn * kPanelBytes, &maps.v[l], pn * 64, kt * kTileN, kvh, b, &bar.v_full[s]);
                    ++issued_v;
                }
            }
            // Before leaving, make sure every copy this lane issued has landed (bounded): the shared
            // memory must not be handed to another CTA with a bulk copy still in flight.
            mbar_wait(&bar.q_full, 0, abortp);
            for (int i = issued_k > C::kStages ? issued_k - C::kStages : 0; i < issued_k; ++i)
                mbar_wait(&bar.k_full[i % C::kStages], (uint32_t)(i / C::kStages) & 1u, abortp);
            for (int i = issued_v > C::kStages ? issued_v - C::kStages : 0; i < issued_v; ++i)
                mbar_wait(&bar.v_full[i % C::kStages], (uint32_t)(i / C::kStages) & 1u, abortp);
        }
    } else if (warp == C::kMmaWarp) {
        {   // every lane runs the issue loop (converged); elect.sync inside the wrappers picks the issuing lane
            bool ok = mbar_wait_warp(&bar.q_full, 0, abortp);
            tc_fence_after();
            // low descriptor words of the operands (see make_desc)
            const uint32_t q_lo = desc_lo_kmajor(smem_u32(sQ)), k_lo = desc_lo_kmajor(smem_u32(sK));
            const uint32_t v_lo = desc_lo_mnmajor(smem_u32(sV), kPanelBytes);
            auto issue_qk = [&](int q, int s) {
                const uint32_t qa = q_lo + q * (C::kTileBytes >> 4), ka = k_lo + s * (C::kTileBytes >> 4);
#pragma unroll
                for (int k = 0; k < DH / 16; ++k)
                    mma_ss_elect(tmem + q * kTileN, make_desc(qa + kstep_off(k, kPanelBytes)), make_desc(ka + kstep_off(k, kPanelBytes)),
                           C::kIdescQK, k > 0);
                mma_commit_elect(&bar.s_full[q]);
            };
            // Paged levels: the page that holds a level's last row is copied whole, so the rows after that row arrive
            // with whatever the pool holds there (a recycled page, never-written memory).  Their weights are exactly 0,
            // but 0 x NaN or 0 x Inf would still poison the accumulator: those V rows are cleared here, after the
            // copy has landed and before the product reads them.  (K needs nothing: masked scores are overwritten.)
            int scrub_e[3] = {-1, -1, -1}, scrub_r0[3] = {0, 0, 0}, scrub_r1[3] = {0, 0, 0};
            if (kPaged) {
                int e0 = 0;
#pragma unroll
                for (int l = 0; l < 3; ++l) {
                    const int tiles = end[l] - first[l];
                    const int tail = (int)(nl[l] % kTileN);
                    if (tiles > 0 && tail != 0 && (long long)end[l] * kTileN > nl[l]) {
                        const int rpb = p.box_rows[l];
                        scrub_e[l] = e0 + tiles - 1;
                        scrub_r0[l] = tail;
                        scrub_r1[l] = (tail + rpb - 1) / rpb * rpb;      // end of the box that straddles the level's end
                    }
                    e0 += tiles;
                }
            }
            auto scrub_v = [&](int e, int s) {
                if constexpr (kPaged) {
#pragma unroll
                for (int l = 0; l < 3; ++l) {
                    if (e != scrub_e[l]) continue;
                    const int vecs = (scrub_r1[l] - scrub_r0[l]) * 8;      // 16-byte vectors per 64-column panel
                    for (int pn = 0; pn < C::kPanels; ++pn) {
                        uint4* base = reinterpret_cast<uint4*>(sV + s * C::kTileBytes + pn * kPanelBytes + scrub_r0[l] * 128);
                        for (int i = lane; i < vecs; i += 32) base[i] = make_uint4(0u, 0u, 0u, 0u);
                    }
                    asm volatile("fence.proxy.async.shared::cta;" ::: "memory");
                    __syncwarp();
                }
                }
            };
            // O_q += P_q V in parts: the softmax warps hand over the weights of 32 keys per thread at a time (K-steps
            // 2 part, 2 part + 1 of every thread's columns), so that the product runs under the remaining exponentials.
            auto issue_pv = [&](int q, int s, int e, bool accumulate) -> bool {
                const uint32_t va = v_lo + s * (C::kTileBytes >> 4);
                const uint32_t pa = tmem + (C::kSeparateP ? C::kColP + q * (kTileN / 2) : q * kTileN);
#pragma unroll
                for (int part = 0; part < C::kParts; ++part) {
                    if (!mbar_wait_warp(&bar.p_part[q][part], (uint32_t)e & 1u, abortp)) return false;
                    tc_fence_after();
#pragma unroll
                    for (int i = 0; i < 2 * C::kSplit; ++i) {
                        const int k = (i >> 1) * (8 / C::kSplit) + part * 2 + (i & 1);
                        mma_ts_elect(tmem + C::kColO + q * DH, pa + k * 8, make_desc(va + k * (2048 >> 4)), C::kIdescPV,
                                     (accumulate || part > 0 || i > 0) ? 1u : 0u);
                    }
                }
                mma_commit_elect(&bar.pv_done[q]);
                return true;
            };
            if (C::kSeparateP) {
                // S_q(e+1) is issued as soon as the warpgroup has S_q(e) in registers; O_q += P_q(e) V(e) when P_q(e) is written.
                if (ok && E > 0) ok = mbar_wait_warp(&bar.k_full[0], 0, abortp);
                if (ok && E > 0) {
                    tc_fence_after();
                    issue_qk(0, 0);
                    issue_qk(1, 0);
                    mma_commit_elect(&bar.k_empty[0]);
                }
                for (int e = 0; e < E && ok; ++e) {
                    const int s = e % C::kStages, sn = (e + 1) % C::kStages;
                    if (e + 1 < E) {
                        if (!mbar_wait_warp(&bar.k_full[sn], (uint32_t)((e + 1) / C::kStages) & 1u, abortp)) { ok = false; break; }
#pragma unroll
                        for (int q = 0; q < C::kNumQ; ++q) {
                            if (!mbar_wait_warp(&bar.s_free[q], (uint32_t)e & 1u, abortp)) { ok = false; break; }
                            tc_fence_after();
                            issue_qk(q, sn);
                        }
                        if (!ok) break;
                        mma_commit_elect(&bar.k_empty[sn]);
                    }
                    if (!mbar_wait_warp(&bar.v_full[s], (uint32_t)(e / C::kStages) & 1u, abortp)) { ok = false; break; }
                    scrub_v(e, s);
#pragma unroll
                    for (int q = 0; q < C::kNumQ; ++q) {
                        if (!issue_pv(q, s, e, e > 0)) { ok = false; break; }
                    }
                    if (!ok) break;
                    mma_commit_elect(&bar.v_empty[s]);
                }
            } else {
            // The wait for K(e+1) is taken before the wait for P_0(e), so that S_0(e+1) follows O_0(e) at once: that
            // pair of products is what query tile 0's softmax threads are waiting for.
            if (ok && E > 0) ok = mbar_wait_warp(&bar.k_full[0], 0, abortp);
            for (int e = 0; e < E && ok; ++e) {
                const int s = e % C::kStages;
                const uint32_t ph = (uint32_t)(e / C::kStages) & 1u;
                tc_fence_after();
                issue_qk(0, s);
                if (e > 0) {
                    const int sp = (e - 1) % C::kStages;
                    if (!issue_pv(1, sp, e - 1, e - 1 > 0)) { ok = false; break; }
                    mma_commit_elect(&bar.v_empty[sp]);
                }
                issue_qk(1, s);
                mma_commit_elect(&bar.k_empty[s]);
                if (!mbar_wait_warp(&bar.v_full[s], ph, abortp)) { ok = false; break; }
                scrub_v(e, s);
                if (e + 1 < E && !mbar_wait_warp(&bar.k_full[(e + 1) % C::kStages], (uint32_t)((e + 1) / C::kStages) & 1u, abortp)) { ok = false; break; }
                if (!issue_pv(0, s, e, e > 0)) { ok = false; break; }
            }
            if (ok && E > 0) {
                const int sp = (E - 1) % C::kStages;
                if (issue_pv(1, sp, E - 1, E - 1 > 0)) mma_commit_elect(&bar.v_empty[sp]);
            }
            }   // !kSeparateP
        }
    }
    } else {
        if constexpr (C::kMoveRegs) asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(C::kRegsSoftmax));
        // ------------------------------------------------------------ softmax warps
        // warp = (query tile, column part, lane quarter); thread = one query row (TMEM lane) x kCols key columns.
        // With two threads per row (d = 64) they agree on the row maximum through shared memory at a 256-thread barrier
        // that also carries their "no wait has run out" flags, so that the 256 threads always leave together.
        const int q = warp / C::kRowWarps, half = (warp >> 2) % C::kSplit;
        const int row_in_tile = (warp & 3) * 32 + lane;
        const int t = (int)m0 + q * kTileM + row_in_tile;    // T < 2^31
        const bool row_valid = t < p.T;
        const uint32_t lane_base = (uint32_t)((warp & 3) * 32) << 16;
        const uint32_t s_addr = tmem + lane_base + q * kTileN + half * C::kCols;
        const uint32_t o_addr = tmem + lane_base + C::kColO + q * DH + half * (DH / C::kSplit);
        // where this thread's weights go as bf16 pairs
        const uint32_t p_addr = (C::kSeparateP ? tmem + lane_base + C::kColP + q * (kTileN / 2) : tmem + lane_base + q * kTileN) + half * (C::kCols / 2);
        const long long tq0 = m0 + (long long)q * kTileM;                      // first row of this query tile
        const long long tq1 = (tq0 + kTileM - 1 < p.T - 1) ? tq0 + kTileM - 1 : p.T - 1;
        auto row_all = [&](bool flag) -> bool {                                 // AND over the threads of the query tile
            if constexpr (C::kSplit == 1) return flag;
            uint32_t out;
            asm volatile("{\n.reg .pred pi, po;\nsetp.ne.u32 pi, %1, 0;\nbar.red.and.pred po, %2, 256, pi;\nselp.u32 %0, 1, 0, po;\n}"
                         : "=r"(out) : "r"((uint32_t)flag), "r"(1 + q) : "memory");
            return out != 0;
        };

        float m_run = -INFINITY, l_run = 0.f;                                    // l_run: this thread's columns only
        bool ok = true, all_ok = true;                                           // ok is warp-uniform
        int e = 0;
        for (int l = 0; l < 3 && all_ok; ++l) {
            if (first[l] == end[l]) continue;
            float bias = -INFINITY;
            int lo = 0, hi = 0;                              // visible rows of this level (levels hold fewer than 2^31 rows)
            if (row_valid) {
                const float g = p.gate[((long long)b * p.T + t) * 3 + l];
                bias = g > 0.f ? log2f(g) : -INFINITY;
                long long lo64, hi64;
                visible_range(l, (long long)t + p.q_offset, p.window, nl[l], 0, lo64, hi64);
                lo = (int)lo64; hi = (int)hi64;
            }
            // key tiles visible to every row of THIS query tile need no element mask
            int full_first = 0, full_end = 0;
            if (tq0 <= tq1) {
                long long lo_f, hi_f, lo_l, hi_l;
                visible_range(l, tq0 + p.q_offset, p.window, nl[l], 0, lo_f, hi_f);
                visible_range(l, tq1 + p.q_offset, p.window, nl[l], 0, lo_l, hi_l);
                full_first = (int)((lo_l + kTileN - 1) / kTileN);
                full_end = (int)(hi_f / kTileN);
                if (tq1 - tq0 + 1 < kTileM) full_end = full_first;         // ragged query tile: always mask
            }
            for (int kt = first[l]; kt < end[l]; ++kt, ++e) {
                if (ok) ok = __all_sync(0xffffffffu, mbar_wait(&bar.s_full[q], (uint32_t)e & 1u, abortp));
                float s[C::kCols];
                float mx = -INFINITY;
                if (ok) {
                    tc_fence_after();
#pragma unroll
                    for (int c0 = 0; c0 < C::kCols; c0 += 32) tmem_ld32(s_addr + c0, reinterpret_cast<uint32_t*>(s) + c0);
                    tmem_ld_wait();
                    if (C::kSeparateP) {                     // S(e) is in registers: its TMEM columns may be reused
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&bar.s_free[q]);
                    }
                    const bool need_mask = !(kt >= full_first && kt < full_end);
                    if (need_mask) {
                        const long long col0 = (long long)kt * kTileN + half * C::kCols;
                        const int c_lo = (int)max(-1LL, min((long long)lo - col0, (long long)C::kCols));
                        const int c_hi = (int)max(-1LL, min((long long)hi - col0, (long long)C::kCols));
#pragma unroll
                        for (int c = 0; c < C::kCols; ++c)
                            if (c < c_lo || c >= c_hi) s[c] = -INFINITY;
                    }
                    float mx4[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
#pragma unroll
                    for (int c = 0; c < C::kCols; c += 8) {
                        mx4[0] = max3(mx4[0], s[c], s[c + 1]); mx4[1] = max3(mx4[1], s[c + 2], s[c + 3]);
                        mx4[2] = max3(mx4[2], s[c + 4], s[c + 5]); mx4[3] = max3(mx4[3], s[c + 6], s[c + 7]);
                    }
                    mx = fmaxf(fmaxf(mx4[0], mx4[1]), fmaxf(mx4[2], mx4[3]));
                }
                if constexpr (C::kSplit == 2) {
                    xmax[e & 1][q][half][row_in_tile] = mx;
                    all_ok = row_all(ok);
                    if (!all_ok) break;
                    mx = fmaxf(mx, xmax[e & 1][q][half ^ 1][row_in_tile]);
                } else {
                    all_ok = ok;
                    if (!all_ok) break;
                }
                const float x_max = fmaf(mx, p.scale_log2, bias);            // -inf when the whole row is masked
                const float m_new = fmaxf(m_run, x_max);
                const bool grow = m_new > m_run + kRescaleThreshold;         // also true for the first finite max
                const float m_use = grow ? m_new : m_run;
                const float m_eff = m_use == -INFINITY ? 0.f : m_use;
                const float alpha = grow ? (m_run == -INFINITY ? 0.f : ex2(m_run - m_use)) : 1.f;
                const float shift = bias - m_eff;
                l_run *= alpha;
                m_run = m_use;
                // P(e-1) must have been consumed before P(e) replaces it (d = 64), and before O is rescaled
                const bool rescale = e > 0 && __any_sync(0xffffffffu, alpha != 1.f);
                if ((C::kSeparateP || rescale) && e > 0) {
                    ok = __all_sync(0xffffffffu, mbar_wait(&bar.pv_done[q], (uint32_t)(e - 1) & 1u, abortp));
                    if (ok) tc_fence_after();
                }
                if (ok) {
                    if (rescale) {                           // some row of this warp moved its reference maximum
#pragma unroll 1
                        for (int c0 = 0; c0 < DH / C::kSplit; c0 += 32) {
                            uint32_t o[32];
                            tmem_ld32(o_addr + c0, o);
                            tmem_ld_wait();
#pragma unroll
                            for (int i = 0; i < 32; ++i) o[i] = __float_as_uint(__uint_as_float(o[i]) * alpha);
                            tmem_st32(o_addr + c0, o);
                        }
                    }
                    // The weights leave in parts of 32 columns (16 packed pairs, one store each).  A part is handed to
                    // the issuing warp in the middle of the next part's exponentials, when its store has long completed.
                    // Scale, shift and the row sum work on packed pairs: one instruction for two columns.
                    const uint64_t scale2 = pack2(p.scale_log2, p.scale_log2), shift2 = pack2(shift, shift);
                    uint64_t sum_a = pack2(0.f, 0.f), sum_b = sum_a;
                    uint32_t pk[16];
                    auto weights = [&](int c_from, int c_to, int c_base) {
#pragma unroll
                        for (int c = c_from; c < c_to; c += 4) {
                            float x0, x1, x2, x3;
                            unpack2(fma2(pack2(s[c], s[c + 1]), scale2, shift2), x0, x1);
                            unpack2(fma2(pack2(s[c + 2], s[c + 3]), scale2, shift2), x2, x3);
                            const float p0 = ex2(x0), p1 = ex2(x1), p2 = ex2(x2), p3 = ex2(x3);
                            sum_a = add2(sum_a, pack2(p0, p1));
                            sum_b = add2(sum_b, pack2(p2, p3));
                            pk[(c - c_base) / 2] = pack_bf16(p0, p1);
                            pk[(c - c_base) / 2 + 1] = pack_bf16(p2, p3);
                        }
                    };
                    auto hand_over = [&](int part) {         // the part (and a rescaled accumulator) is in TMEM
                        tmem_st_wait();
                        tc_fence_before();
                        __syncwarp();
                        if (lane == 0) mbar_arrive(&bar.p_part[q][part]);
                    };
#pragma unroll
                    for (int part = 0; part < C::kParts; ++part) {
                        weights(32 * part, 32 * part + 16, 32 * part);
                        if (part > 0) hand_over(part - 1);
                        weights(32 * part + 16, 32 * part + 32, 32 * part);
                        tmem_st16(p_addr + 16 * part, pk);
                    }
                    {
                        float a0, a1;
                        unpack2(add2(sum_a, sum_b), a0, a1);
                        l_run += a0 + a1;
                    }
                    hand_over(C::kParts - 1);
                }
            }
        }
        // ------------------------------------------------------------ epilogue
        if (all_ok) {
            if (ok && E > 0) ok = __all_sync(0xffffffffu, mbar_wait(&bar.pv_done[q], (uint32_t)(E - 1) & 1u, abortp));
            if constexpr (C::kSplit == 2) lsum[q][half][row_in_tile] = l_run;   // the row's sum is the sum of its two halves
            all_ok = row_all(ok);
        }
        if (all_ok) {
            tc_fence_after();
            float l_row = l_run;
            if constexpr (C::kSplit == 2) l_row += lsum[q][half ^ 1][row_in_tile];
            const float inv = l_row > 0.f ? 1.f / l_row : 0.f;   // rows with nothing visible: exact zeros
            __nv_bfloat16* Orow = p.O + (((long long)b * p.H + h) * p.T + t) * DH + half * (DH / C::kSplit);
#pragma unroll 1
            for (int c0 = 0; c0 < DH / C::kSplit; c0 += 32) {
                uint32_t o[32];
                if (E > 0) {
                    tmem_ld32(o_addr + c0, o);
                    tmem_ld_wait();
                } else {
#pragma unroll
                    for (int i = 0; i < 32; ++i) o[i] = 0u;
                }
                if (row_valid) {
#pragma unroll
                    for (int i = 0; i < 32; i += 8) {
                        uint4 v;
                        const float z = inv;
                        v.x = pack_bf16(z > 0.f ? __uint_as_float(o[i]) * z : 0.f, z > 0.f ? __uint_as_float(o[i + 1]) * z : 0.f);
                        v.y = pack_bf16(z > 0.f ? __uint_as_float(o[i + 2]) * z : 0.f, z > 0.f ? __uint_as_float(o[i + 3]) * z : 0.f);
                        v.z = pack_bf16(z > 0.f ? __uint_as_float(o[i + 4]) * z : 0.f, z > 0.f ? __uint_as_float(o[i + 5]) * z : 0.f);
                        v.w = pack_bf16(z > 0.f ? __uint_as_float(o[i + 6]) * z : 0.f, z > 0.f ? __uint_as_float(o[i + 7]) * z : 0.f);
                        *reinterpret_cast<uint4*>(Orow + c0 + i) = v;
                    }
                }
            }
            if (row_valid && half == 0 && p.LSE)
                p.LSE[((long long)b * p.H + h) * p.T + t] = l_row > 0.f ? (m_run + log2f(l_row)) * kLn2 : -INFINITY;
        }
    }

    tc_fence_before();
    __syncthreads();
    if (tid == 0 && wait_ctl.abort) atomicExch(p.status, (unsigned int)MKA_ERR_TIMEOUT);
    if (warp == 0) asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(C::kTmemCols) : "memory");
}

inline bool make_map(CUtensorMap* map, const void* base, int d, long long rows, int H, int B, long long sn, long long sh, long long sb) {
    return make_bf16_map(map, base, d, rows, H, B, sn, sh, sb, 128);
}

template <int DH>
cudaError_t launch_t(const FwdParams& fp, unsigned int* status_word, cudaStream_t st) {
    TcMaps maps;
    if (!make_map(&maps.q, fp.Q, DH, fp.T, fp.H, fp.B, DH, (long long)fp.T * DH, (long long)fp.H * fp.T * DH))
        return cudaErrorNotSupported;
    TcParams p;
    memset(&p, 0, sizeof(p));
    p.paged = fp.paged ? 1 : 0;
    for (int l = 0; l < 3; ++l) {
        if (fp.L[l].n == 0) { maps.k[l] = maps.q; maps.v[l] = maps.q; continue; }
        if (fp.paged) {
            // the pool as a [pages, KV heads, rows of a page, d] tensor; a box = (up to 128) rows of one page
            const PagedLevelDev& P = fp.paged[l];
            const int page_rows = 1 << P.page_shift;
            const int rpb = page_rows < kTileN ? page_rows : kTileN;
            if (!make_bf16_map(&maps.k[l], P.k, DH, page_rows, fp.H / fp.kv_group, (int)P.pool_pages, P.sn, P.sh, P.sp, rpb) ||
                !make_bf16_map(&maps.v[l], P.v, DH, page_rows, fp.H / fp.kv_group, (int)P.pool_pages, P.sn, P.sh, P.sp, rpb))
                return cudaErrorNotSupported;
            p.table[l] = P.table; p.table_stride[l] = P.table_stride; p.table_head_stride[l] = P.table_head_stride;
            p.page_shift[l] = P.page_shift; p.box_rows[l] = rpb; p.pool_pages[l] = (int)P.pool_pages; p.rows[l] = P.rows;
            continue;
        }
        if (!make_map(&maps.k[l], fp.L[l].k, DH, fp.L[l].n, fp.H / fp.kv_group, fp.B, fp.L[l].sn, fp.L[l].sh, fp.L[l].sb) ||
            !make_map(&maps.v[l], fp.L[l].v, DH, fp.L[l].n, fp.H / fp.kv_group, fp.B, fp.L[l].sn, fp.L[l].sh, fp.L[l].sb))
            return cudaErrorNotSupported;
    }
    p.O = static_cast<__nv_bfloat16*>(fp.O);
    p.LSE = fp.LSE;
    p.gate = fp.gate;
    for (int l = 0; l < 3; ++l) p.n[l] = fp.L[l].n;
    p.B = fp.B; p.H = fp.H; p.T = fp.T; p.kv_group = fp.kv_group;
    p.window = fp.window; p.q_offset = fp.q_offset;
    p.scale_log2 = fp.scale * kLog2e;
    p.status = status_word;
    p.wait_limit_ns = wait_limit_ns();
    p.test_stall = fp.test_stall;
    {   // as many (batch, head) pairs per group as keep the group's K and V (48 MB at most) in the L2 cache while
        // its blocks, dealt by query block, re-read them
        double pair_bytes = 0.0;
        for (int l = 0; l < 3; ++l) pair_bytes += (double)fp.L[l].n * DH * 4.0;
        pair_bytes /= fp.kv_group;
        const double pairs = (double)fp.B * fp.H;
        const double fit = pair_bytes > 0.0 ? 48.0 * 1024 * 1024 / pair_bytes : pairs;
        p.deal = fit < 1.0 ? 1 : (fit > pairs ? (int)pairs : (int)fit);
    }
    auto kern = fp.paged ? fwd_tc_kernel<DH, true> : fwd_tc_kernel<DH, false>;
    cudaError_t e = cudaFuncSetAttribute(kern, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)Cfg<DH>::kSmemBytes);
    if (e != cudaSuccess) return e;
    dim3 grid((fp.T + Cfg<DH>::kNumQ * kTileM - 1) / (Cfg<DH>::kNumQ * kTileM), fp.H, fp.B);
    kern<<<grid, Cfg<DH>::kThreads, Cfg<DH>::kSmemBytes, st>>>(maps, p);
    return cudaGetLastError();
}

}  // namespace

bool fwd_tc_eligible(const FwdParams& p, int dtype) {
    if (dtype != MKA_BF16 || p.mode != MKA_MODE_FAST || p.decode) return false;
    if (p.d != 64 && p.d != 128) return false;
    if (p.H > 65535 || p.B > 65535) return false;
    if ((double)((p.T + 127) / 128) * p.H * p.B > 2147483647.0) return false;   // the kernel numbers its blocks in an int
    for (int l = 0; l < 3; ++l) {
        const LevelDev& L = p.L[l];
        if (L.n == 0) continue;
        if (L.n > 0x7fffffffLL) return false;
        if (L.sn % 8 || L.sn <= 0) return false;
        if (p.H / (p.kv_group > 0 ? p.kv_group : 1) > 1 && (L.sh % 8 || L.sh <= 0)) return false;
        if (p.B > 1 && (L.sb % 8 || L.sb <= 0)) return false;
    }
    return tensor_map_encoder_available();
}

cudaError_t launch_fwd_tc(const FwdParams& p, unsigned int* status_word, cudaStream_t st) {
    if (p.B == 0 || p.H == 0 || p.T == 0) return cudaSuccess;
    return p.d == 128 ? launch_t<128>(p, status_word, st) : launch_t<64>(p, status_word, st);
}

}  // namespace mka
