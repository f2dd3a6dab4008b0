// Block-sparse attention forward on the 5th-generation tensor cores (tcgen05 + TMEM + TMA).
//
// Formulation.  The selection is per 64-row query block, but the tensor-core datapath is 128 rows
// high and a K/V tile costs as much shared-memory bandwidth to stage as to multiply.  One CTA
// therefore owns TWO query blocks (rows 0-63 = block A, rows 64-127 = block B of one head) and
// walks the ascending UNION of their two key-block lists, two key blocks (128 keys) per tile:
//
//     S[128 q x 128 keys]  = Q . K_tile^T      tcgen05.mma, A = Q in smem,        B = K in smem
//     O[128 q x 128 d]    += P . V_tile        tcgen05.mma, A = P (bf16) in TMEM, B = V in smem
//
// A key block that only one of the two lists holds is masked for the other half of the rows
// (its softmax weights are written as zero), so the result is exactly the per-block selection.
// Nearby query blocks of video tokens select largely the same key blocks, which is what makes
// the shared tile pay; which two blocks share a CTA is chosen per call for large list overlap
// (usv_attn_plan.cu).
//
// Query rows live on TMEM lanes: softmax thread i owns row i, so maxima and sums need no
// cross-thread traffic.  The softmax reference of a row (the value subtracted inside the
// exponential) is fixed at the row maximum over the first key block the row may see and never
// changes, so O needs no rescaling; the exponent range of fp32/bf16 absorbs later, larger
// logits.  Rows whose sum leaves [2^-100, 2^100] are reported in a list and recomputed by the
// exact online-softmax kernel, so the result never depends on that assumption.
//
// CTA = 19 warps.  Warps 0-15 are four softmax/epilogue warpgroups that share the 128 rows
// (thread r of every group <-> TMEM lane r <-> query row r).  Group g works on the tiles of
// parity g >> 1 and there on key block g & 1 of the tile (64 logit columns), so two tiles are in
// the softmax stage at a time, each spread over 256 threads.  Warp 16 is the K producer (TMA; it
// also fetches the pair's Q rows), warp 17 the MMA issuer and TMEM owner, warp 18 the V producer.
//
// TMEM holds O and THREE S buffers; tile t uses buffer t mod 3.  The weights P(t) are written
// back, as bf16 pairs, into the columns their logits came from, so a buffer goes
// S(t) -> P(t) -> S(t + 3) without a hand-back: P.V(t) is issued before S(t + 3), and the tensor
// pipe runs its MMAs in issue order.  With three buffers a finished S tile is always waiting
// when a softmax group comes free, and a finished P tile when the pipe does.  Every barrier has
// one set of waiters that sees each of its phases (SFULL/PFULL are indexed by t mod 6: the two
// tile parities of a buffer wait on different barriers; a waiter that skipped a phase could not
// tell it from the one two before).  All waits are bounded; a wait that gives up sets the device
// status word and every role leaves its loop.
#include "usv_attn.cuh"
#include "usv_tcgen05.cuh"

namespace usv {

namespace pr {

using namespace t5;

constexpr int D = 128;
constexpr int KT = 2 * USV_BLOCK;               // keys per tile = two key blocks
constexpr int NWG = 4;                          // softmax warpgroups
constexpr int KSTAGES = 2;                      // K tile stages
constexpr int VSTAGES = 3;                      // V tile stages
constexpr int MAX_NB = 4096;                    // key blocks per sequence this kernel covers
constexpr uint32_t TILE_BYTES = KT * D * 2;     // 32 KB: [d-half][128 keys][128 B]
constexpr int SBUF = 3;                         // S/P buffers in TMEM
constexpr uint32_t SM_Q = 0;                    // the pair's 128 query rows, same layout as a K tile
constexpr uint32_t SM_K = SM_Q + TILE_BYTES;
constexpr uint32_t SM_V = SM_K + KSTAGES * TILE_BYTES;
constexpr uint32_t SM_BAR = SM_V + VSTAGES * TILE_BYTES;
// barrier slots (8 bytes each)
enum { B_QFULL = 0, B_KFULL = 1, B_KEMPTY = B_KFULL + KSTAGES, B_VFULL = B_KEMPTY + KSTAGES,
       B_VEMPTY = B_VFULL + VSTAGES, B_SFULL = B_VEMPTY + VSTAGES, B_PFULL = B_SFULL + 2 * SBUF,
       B_OFULL = B_PFULL + 2 * SBUF, B_REF, B_EPI = B_REF + 2, B_COUNT = B_EPI + 2 };
static_assert(B_COUNT <= 32, "barrier area");
constexpr uint32_t SM_MISC = SM_BAR + 8 * 32;            // tmem base, abort flag, flags, union size
constexpr uint32_t SM_LIST = SM_MISC + 64;               // int[MAX_NB]: (key block << 2) | in-A | in-B << 1
constexpr uint32_t SM_REFV = SM_LIST + MAX_NB * 4;       // float[128]: minus the softmax reference per row
constexpr uint32_t SM_SUM = SM_REFV + 128 * 4;           // float[NWG][128]: partial row sums
constexpr uint32_t SM_TOTAL = SM_SUM + NWG * 128 * 4;
constexpr size_t SMEM_BYTES = SM_TOTAL + 1024;           // + slack for 1024-byte alignment

// TMEM columns: O | S/P buffer 0 | S/P buffer 1 | S/P buffer 2
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t TO = 0, TS = 128;
static_assert(TS + SBUF * 128 <= TMEM_COLS, "TMEM budget");

constexpr int NSOFT = NWG * 128;   // softmax threads
constexpr int NTHREADS = NSOFT + 96;
constexpr int W_TMA = NSOFT / 32, W_MMA = NSOFT / 32 + 1, W_TMA_V = NSOFT / 32 + 2;

struct Maps {
    CUtensorMap q, k, v;
};

// exp2 of 32 scaled logits -> 16 packed bf16 pairs; adds the weights, as rounded to bf16 (what
// the P.V product multiplies by), to the two lanes of `acc`, so that numerator and denominator of
// a row carry the same rounding.  Two logits at a time on the packed-fp32 pipe.
template <bool MASKED>
__device__ __forceinline__ void weights32(const uint32_t* sr, uint32_t* pk, uint64_t c2, uint64_t nref2, int col0,
                                          int nvalid, uint64_t& acc) {
#pragma unroll
    for (int j = 0; j < 16; ++j) {
        const uint64_t x2 = fma_f32x2(pack_f32x2(__uint_as_float(sr[2 * j]), __uint_as_float(sr[2 * j + 1])), c2, nref2);
        float x0, x1;
        unpack_f32x2(x2, x0, x1);
        float p0 = ex2(x0), p1 = ex2(x1);
        if (MASKED) {
            if (col0 + 2 * j >= nvalid) p0 = 0.f;
            if (col0 + 2 * j + 1 >= nvalid) p1 = 0.f;
        }
        pk[j] = pack_bf16x2(p0, p1);
        acc = add_f32x2(acc, pack_f32x2(__uint_as_float(pk[j] << 16), __uint_as_float(pk[j] & 0xffff0000u)));
    }
}

__global__ void __launch_bounds__(NTHREADS, 1)
attn_pair_kernel(const AttnArgs a, const __grid_constant__ Maps maps) {
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* sm = smem_raw + (base - raw);
    auto bar = [&](int i) { return base + SM_BAR + 8u * i; };
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(sm + SM_MISC);
    volatile int* s_abort = reinterpret_cast<volatile int*>(sm + SM_MISC + 4);
    volatile int* s_flag = reinterpret_cast<volatile int*>(sm + SM_MISC + 8);   // [2]
    volatile int* s_nu = reinterpret_cast<volatile int*>(sm + SM_MISC + 16);
    int* s_list = reinterpret_cast<int*>(sm + SM_LIST);
    float* s_refv = reinterpret_cast<float*>(sm + SM_REFV);
    float* s_sum = reinterpret_cast<float*>(sm + SM_SUM);

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int NB = a.NB, N = a.N;
    const int NP = (NB + 1) >> 1;                 // query-block pairs per (b, h)
    const int pair = blockIdx.x % NP;
    const int bh_ord = blockIdx.x / NP;
    const int b = bh_ord / a.H;
    const int h = a.head_order[bh_ord % a.H];
    const int kh = a.k_per_head[h];
    const int2 pq = a.pairs[((int64_t)b * a.H + h) * NP + pair];   // similarity-driven pairing
    const int IA = pq.x;
    const int IB = pq.y;

    // softmax-thread geometry (meaningful for warps < W_TMA)
    const int grp = warp >> 2;                       // tiles of parity grp >> 1, key block grp & 1
    const int r = threadIdx.x & 127;                 // query row within the pair, = TMEM lane
    const int side = r >> 6;                         // 0: block A, 1: block B (uniform per warp)
    const int Iq = side ? IB : IA;
    const int row = Iq * USV_BLOCK + (r & 63);
    const bool live = Iq >= 0 && row < N;

    // ---- set-up: barriers, TMEM, the pair's key-block list -> shared memory
    if (warp == 0) {
        // one barrier per lane (a single thread initialising all of them takes ~1000 cycles)
        uint32_t count = 1;                                           // Q, K/V stages, SFULL, OFULL
        if (lane == B_EPI || lane == B_EPI + 1) count = NSOFT / 32;   // one arrival per softmax warp
        // PFULL: one arrival per warp of the two groups of a tile
        if (lane >= B_PFULL && lane < B_PFULL + 2 * SBUF) count = 8;
        // REF / EPI: rendezvous of the softmax threads after the first bounded wait: mbarriers, so
        // that they too can give up (a bar.sync would hang if one thread had left its loop)
        if (lane == B_REF || lane == B_REF + 1) count = 2;            // the two warps of the owning group on a side
        if (lane < B_COUNT) mbar_init(bar(lane), count);
        if (lane == 0) {
            *s_abort = 0;
            s_flag[0] = 0;
            s_flag[1] = 0;
        }
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == W_MMA) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(base + SM_MISC), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    const int* plist = a.lists + b * a.list_batch + a.list_off[h] + (int64_t)pair * list_stride(kh, NB);
    if (warp < W_TMA) {
        // the pair's union key-block list (built by the plan kernels) -> shared memory
        const int lstride = (int)list_stride(kh, NB);
        for (int i = threadIdx.x; i < lstride; i += NSOFT) {
            const int e = plist[i];
            if (i == 0) *s_nu = e; else s_list[i - 1] = e;
        }
    }
    fence_before();
    __syncthreads();
    fence_after();
    const uint32_t tmem = *s_tmem;
    const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
    const int nU = *s_nu;
    const int T = (nU + 1) >> 1;   // 128-key tiles

    if (warp == W_TMA) {
        // ===== K producer (whole warp in the loop, one elected lane issues) =====================
        // K and V have a producer warp each: a K stage comes back as soon as S is computed, long
        // before the V stage of the same tile does, and must not queue behind it.
        if (T > 0 && elect_one()) {
            // the pair's query rows; a block without a partner reads rows past the end (zero fill)
            const int ra = IA * USV_BLOCK, rb = (IB >= 0 ? IB : NB) * USV_BLOCK;
            mbar_expect_tx(bar(B_QFULL), TILE_BYTES);
            tma_load_4d(base + SM_Q, &maps.q, bar(B_QFULL), 0, ra, h, b);
            tma_load_4d(base + SM_Q + 8192, &maps.q, bar(B_QFULL), 0, rb, h, b);
            tma_load_4d(base + SM_Q + 16384, &maps.q, bar(B_QFULL), 64, ra, h, b);
            tma_load_4d(base + SM_Q + 24576, &maps.q, bar(B_QFULL), 64, rb, h, b);
        }
        __syncwarp();
        for (int t = 0; t < T; ++t) {
            const int s = t % KSTAGES;
            const uint32_t ph = (t / KSTAGES) & 1;
            const int J0 = s_list[2 * t] >> 2;
            const int J1 = (2 * t + 1 < nU) ? (s_list[2 * t + 1] >> 2) : J0;  // odd tail: finite filler, masked
            if (!mbar_wait(bar(B_KEMPTY + s), ph ^ 1, s_abort, a.status, 0x1)) break;
            const uint32_t kd = base + SM_K + s * TILE_BYTES;
            if (elect_one()) {
                mbar_expect_tx(bar(B_KFULL + s), TILE_BYTES);
                tma_load_4d(kd, &maps.k, bar(B_KFULL + s), 0, J0 * USV_BLOCK, h, b);
                tma_load_4d(kd + 8192, &maps.k, bar(B_KFULL + s), 0, J1 * USV_BLOCK, h, b);
                tma_load_4d(kd + 16384, &maps.k, bar(B_KFULL + s), 64, J0 * USV_BLOCK, h, b);
                tma_load_4d(kd + 24576, &maps.k, bar(B_KFULL + s), 64, J1 * USV_BLOCK, h, b);
            }
            __syncwarp();
        }
    } else if (warp == W_TMA_V) {
        // ===== V producer =======================================================================
        for (int t = 0; t < T; ++t) {
            const int sv = t % VSTAGES;
            const uint32_t phv = (t / VSTAGES) & 1;
            const int J0 = s_list[2 * t] >> 2;
            const int J1 = (2 * t + 1 < nU) ? (s_list[2 * t + 1] >> 2) : J0;
            if (!mbar_wait(bar(B_VEMPTY + sv), phv ^ 1, s_abort, a.status, 0x2)) break;
            const uint32_t vd = base + SM_V + sv * TILE_BYTES;
            if (elect_one()) {
                mbar_expect_tx(bar(B_VFULL + sv), TILE_BYTES);
                tma_load_4d(vd, &maps.v, bar(B_VFULL + sv), 0, J0 * USV_BLOCK, h, b);
                tma_load_4d(vd + 8192, &maps.v, bar(B_VFULL + sv), 0, J1 * USV_BLOCK, h, b);
                tma_load_4d(vd + 16384, &maps.v, bar(B_VFULL + sv), 64, J0 * USV_BLOCK, h, b);
                tma_load_4d(vd + 24576, &maps.v, bar(B_VFULL + sv), 64, J1 * USV_BLOCK, h, b);
            }
            __syncwarp();
        }
    } else if (warp == W_MMA) {
        // ===== MMA issuer (whole warp in the loop, one elected lane issues); TMEM owner =========
        if (T > 0) {
            constexpr uint32_t IDESC_S = instr_desc(128, KT, 0, 0);    // Q (K-major) x K (K-major)
            constexpr uint32_t IDESC_O = instr_desc(128, D, 0, 1);     // P (TMEM) x V (MN-major)
            const uint64_t qdesc0 = smem_desc(base + SM_Q, 16, 1024);       // + byte offset >> 4
            const uint64_t kdesc0 = smem_desc(base + SM_K, 16, 1024);
            const uint64_t vdesc0 = smem_desc(base + SM_V, 16384, 1024);
            bool ok = mbar_wait(bar(B_QFULL), 0, s_abort, a.status, 0x4);
            // S(t) -> buffer t % SBUF.  The buffer's previous tenant, P(t - SBUF), is read by
            // PV(t - SBUF), which was issued before: the tensor pipe runs its MMAs in issue order.
            auto issue_s = [&](int t, bool k_ready) -> bool {
                const int s = t % KSTAGES;
                const uint32_t ph = (t / KSTAGES) & 1;
                if (!k_ready && !mbar_wait(bar(B_KFULL + s), ph, s_abort, a.status, 0x8)) return false;
                fence_after();
                const uint64_t kdesc = kdesc0 + ((s * TILE_BYTES) >> 4);
                const uint32_t d_s = tmem + TS + (t % SBUF) * 128;
                if (elect_one()) {
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks) {
                        const uint32_t off = ((ks >> 2) * 16384 + (ks & 3) * 32) >> 4;
                        umma_ss(d_s, qdesc0 + off, kdesc + off, IDESC_S, ks > 0);
                    }
                    umma_commit(bar(B_SFULL + t % (2 * SBUF)));
                }
                return true;
            };
            for (int t = 0; ok && t < SBUF && t < T; ++t) ok = issue_s(t, false);
            for (int t = 0; ok && t < T; ++t) {
                const int sv = t % VSTAGES;
                const uint32_t phv = (t / VSTAGES) & 1;
                const int sb6 = t % (2 * SBUF);
                const uint32_t php = (t / (2 * SBUF)) & 1;
                // poll the barriers of this step together: their latencies overlap
                const int t3 = t + SBUF;
                const bool k_rdy = t3 < T && mbar_try(bar(B_KFULL + t3 % KSTAGES), (t3 / KSTAGES) & 1);
                const bool v_rdy = mbar_try(bar(B_VFULL + sv), phv);
                const bool p_rdy = mbar_try(bar(B_PFULL + sb6), php);
                if (!v_rdy && !mbar_wait(bar(B_VFULL + sv), phv, s_abort, a.status, 0x20)) break;
                if (!p_rdy && !mbar_wait(bar(B_PFULL + sb6), php, s_abort, a.status, 0x40)) break;
                fence_after();
                const uint64_t vdesc = vdesc0 + ((sv * TILE_BYTES) >> 4);
                const uint32_t pb = tmem + TS + (t % SBUF) * 128;   // P(t): 32 columns at the head of each 64-column half
                if (elect_one()) {
#pragma unroll
                    for (int ks = 0; ks < KT / 16; ++ks)
                        umma_ts(tmem + TO, pb + (ks >> 2) * 64 + (ks & 3) * 8, vdesc + ((ks * 2048) >> 4), IDESC_O,
                                (t > 0 || ks > 0));
                    umma_commit(bar(B_VEMPTY + sv));
                    if (t == T - 1) umma_commit(bar(B_OFULL));
                }
                __syncwarp();
                if (t3 < T) ok = issue_s(t3, k_rdy);
            }
        }
    } else if (T > 0) {
        // ===== softmax + epilogue =====
        const float c = a.scale_log2;
        // First union slot whose key block this row may see (lists only, so uniform over the
        // query block): the group that owns that slot fixes the row's softmax reference there
        // and publishes it; the other groups pick it up before their first later slot.
        int sref = nU;
        for (int sl = 0; sl < nU; ++sl)
            if ((s_list[sl] >> side) & 1) { sref = sl; break; }
        const int tp = grp >> 1, hb = grp & 1;
        float nref = 0.f;         // minus the softmax reference (base-2, scaled)
        bool have_ref = false;
        uint64_t lr2 = 0;         // two partial sums of the weights this thread produced for its row
        uint64_t nref2 = 0;
        const uint64_t c2 = pack_f32x2(c, c);
        bool ok = true;
        const bool releaser = hb == 0 && (warp & 3) == 0 && lane == 0;   // hands K stages back
        for (int t = tp; t < T; t += 2) {
            const int slot = 2 * t + hb;
            const int e = slot < nU ? s_list[slot] : 0;
            const bool mine = (e >> side) & 1;
            const int nv = N - (e >> 2) * USV_BLOCK;   // keys of the block with index < N
            const uint32_t sbase = lane_base + TS + (t % SBUF) * 128 + hb * 64;
            if (!mbar_wait(bar(B_SFULL + t % (2 * SBUF)), (t / (2 * SBUF)) & 1, s_abort, a.status, 0x80)) { ok = false; break; }
            fence_after();
            if (releaser) mbar_arrive(bar(B_KEMPTY + t % KSTAGES));   // S(t) is complete
            if (!have_ref && slot >= sref) {
                if (slot == sref) {
                    // one-off pass over this key block for the row maximum (the block is mine here)
                    uint32_t m0[32], m1[32];
                    tmem_ld32(sbase, m0);
                    tmem_ld32(sbase + 32, m1);
                    tmem_wait_ld();
                    float mx = -INFINITY;
#pragma unroll
                    for (int j = 0; j < 32; ++j) {
                        if (j < nv) mx = fmaxf(mx, __uint_as_float(m0[j]));
                        if (j + 32 < nv) mx = fmaxf(mx, __uint_as_float(m1[j]));
                    }
                    nref = mx == -INFINITY ? 0.f : -mx * c;
                    s_refv[r] = nref;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(B_REF + side));
                } else {
                    if (!mbar_wait(bar(B_REF + side), 0, s_abort, a.status, 0x400)) { ok = false; break; }
                    nref = s_refv[r];
                }
                nref2 = pack_f32x2(nref, nref);
                have_ref = true;
            }
            // The weights (bf16 pairs) go back into the columns their logits came from: P(t) takes
            // the first 32 of the 64 columns, each half written once its logits are in registers.
            uint32_t pk0[16], pk1[16];
            if (mine) {
                uint32_t sx[32];
                tmem_ld32(sbase, sx);
                tmem_wait_ld();
                if (nv >= USV_BLOCK) weights32<false>(sx, pk0, c2, nref2, 0, nv, lr2);
                else weights32<true>(sx, pk0, c2, nref2, 0, nv, lr2);
                tmem_ld32(sbase + 32, sx);
                tmem_wait_ld();
                tmem_st16(sbase, pk0);
                if (nv >= USV_BLOCK) weights32<false>(sx, pk1, c2, nref2, 32, nv, lr2);
                else weights32<true>(sx, pk1, c2, nref2, 32, nv, lr2);
                tmem_st16(sbase + 16, pk1);
            } else {
#pragma unroll
                for (int j = 0; j < 16; ++j) pk0[j] = 0u;
                tmem_st16(sbase, pk0);
                tmem_st16(sbase + 16, pk0);
            }
            tmem_wait_st();
            fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(B_PFULL + t % (2 * SBUF)));
        }
        // ---- epilogue
        if (ok) ok = mbar_wait(bar(B_OFULL), 0, s_abort, a.status, 0x200);
        if (ok) {
            fence_after();
            float lr_lo, lr_hi;
            unpack_f32x2(lr2, lr_lo, lr_hi);
            s_sum[grp * 128 + r] = lr_lo + lr_hi;
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(B_EPI));
            ok = mbar_wait(bar(B_EPI), 0, s_abort, a.status, 0x800);
        }
        if (ok) {
            float l = 0.f;
#pragma unroll
            for (int g = 0; g < NWG; ++g) l += s_sum[g * 128 + r];
            const bool in_range = l > 7.9e-31f && l < 1.2e30f;   // ~[2^-100, 2^100]
            if (live && !in_range) s_flag[side] = 1;
            const float inv = l > 0.f ? 1.0f / l : 0.f;
            if (a.lse != nullptr && live && grp == 0)
                a.lse[((int64_t)b * a.H + h) * N + row] =
                    (log2f(l) - (sref < nU ? s_refv[r] : 0.f)) * 0.69314718055994531f;
            float* o32 = (a.o_f32 != nullptr && live)
                             ? a.o_f32 + (((int64_t)b * a.H + h) * N + row) * D + grp * 32 : nullptr;
            unsigned char* stage = sm + SM_V;   // [128 rows][256 B], 16-byte chunks XOR-swizzled by row
            uint32_t orr[32];
            tmem_ld32(lane_base + TO + grp * 32, orr);
            tmem_wait_ld();
            float f[32];
#pragma unroll
            for (int j = 0; j < 32; ++j) f[j] = __uint_as_float(orr[j]) * inv;
            if (o32 != nullptr) {
#pragma unroll
                for (int j = 0; j < 8; ++j)
                    *reinterpret_cast<float4*>(o32 + j * 4) = make_float4(f[4 * j], f[4 * j + 1], f[4 * j + 2], f[4 * j + 3]);
            }
#pragma unroll
            for (int i = 0; i < 4; ++i) {
                const int cc = grp * 4 + i;
                *reinterpret_cast<uint4*>(stage + r * 256 + ((cc ^ (r & 15)) << 4)) = float8_to_bf16x8(f + 8 * i);
            }
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(B_EPI + 1));
            ok = mbar_wait(bar(B_EPI + 1), 0, s_abort, a.status, 0x1000);
        }
        if (ok) {
            unsigned char* stage = sm + SM_V;
            __nv_bfloat16* O = a.o + b * a.so.sb + h * a.so.sh;
#pragma unroll 4
            for (int idx = threadIdx.x; idx < 128 * 16; idx += NSOFT) {
                const int rr = idx >> 4, cc = idx & 15;
                const int Ir = rr < 64 ? IA : IB;
                const int grow = Ir * USV_BLOCK + (rr & 63);
                if (Ir >= 0 && grow < N)
                    *reinterpret_cast<uint4*>(O + (int64_t)grow * a.so.sn + cc * 8) =
                        *reinterpret_cast<const uint4*>(stage + rr * 256 + ((cc ^ (rr & 15)) << 4));
            }
        }
    }

    // ---- teardown
    fence_before();
    __syncthreads();
    if (*s_abort) {
        // give copies and MMAs that may still be in flight time to land before the CTA's
        // shared memory and TMEM are handed back
        const unsigned long long t0 = gtime();
        while (gtime() - t0 < 2000000ull) { }
        __syncthreads();
    }
    if (threadIdx.x < 2 && T > 0 && s_flag[threadIdx.x] && a.fallback_list != nullptr) {
        const int slot = atomicAdd(a.fallback_count, 1);
        a.fallback_list[slot] = bh_ord * NB + (threadIdx.x ? IB : IA);
    }
    if (T == 0) {
        // no valid key block at all: defined output (zeros, log-sum-exp 0), as the exact kernel does
        __nv_bfloat16* O = a.o + b * a.so.sb + h * a.so.sh;
        for (int idx = threadIdx.x; idx < 128 * (D / 8); idx += blockDim.x) {
            const int rr = idx / (D / 8), cc = idx % (D / 8);
            const int Ir = rr < 64 ? IA : IB;
            const int grow = Ir * USV_BLOCK + (rr & 63);
            if (Ir >= 0 && grow < N) {
                *reinterpret_cast<uint4*>(O + (int64_t)grow * a.so.sn + cc * 8) = make_uint4(0, 0, 0, 0);
                const int64_t grow_bh = ((int64_t)b * a.H + h) * N + grow;
                if (a.o_f32 != nullptr) {
                    float4* o32 = reinterpret_cast<float4*>(a.o_f32 + grow_bh * D + cc * 8);
                    o32[0] = make_float4(0.f, 0.f, 0.f, 0.f);
                    o32[1] = make_float4(0.f, 0.f, 0.f, 0.f);
                }
                if (a.lse != nullptr && cc == 0) a.lse[grow_bh] = 0.f;
            }
        }
    }
    if (warp == W_MMA) {
        fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
    }
}

}  // namespace pr

bool attn_pair_supported(const AttnArgs& a, int d) {
    return d == pr::D && a.NB <= pr::MAX_NB;
}

int launch_attn_pair(const AttnArgs& a, int d, cudaStream_t st) {
    pr::Maps maps;
    int rc;
    if ((rc = t5::make_bhnd_map(&maps.q, a.q, a.sq, a.B, a.H, a.N, d, "q")) != USV_OK) return rc;
    if ((rc = t5::make_bhnd_map(&maps.k, a.k, a.sk, a.B, a.H, a.N, d, "k")) != USV_OK) return rc;
    if ((rc = t5::make_bhnd_map(&maps.v, a.v, a.sv, a.B, a.H, a.N, d, "v")) != USV_OK) return rc;
    const int64_t grid = (int64_t)a.B * a.H * ((a.NB + 1) / 2);
    if (grid > 2147483647LL) return fail(USV_ERR_UNSUPPORTED, "sparse_attn: too many query blocks");
    cudaError_t e = cudaFuncSetAttribute(pr::attn_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)pr::SMEM_BYTES);
    if (e != cudaSuccess) return fail(USV_ERR_CUDA, "sparse_attn: smem attribute: %s", cudaGetErrorString(e));
    pr::attn_pair_kernel<<<(unsigned)grid, pr::NTHREADS, pr::SMEM_BYTES, st>>>(a, maps);
    USV_CHECK_LAUNCH("attn_pair_kernel");
    return USV_OK;
}

}  // namespace usv
