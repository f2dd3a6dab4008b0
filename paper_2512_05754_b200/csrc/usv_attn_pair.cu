// Block-sparse attention forward on the 5th-generation tensor cores (tcgen05 + TMEM + TMA).
//
// Formulation.  The selection is per 64-row query block, but the tensor-core datapath is 128 rows
// high and a K/V tile costs as much shared-memory bandwidth to stage as to multiply.  One work
// item is therefore a PAIR of query blocks of one head (rows 0-63 = block A, rows 64-127 =
// block B) and walks the ascending UNION of their two key-block lists, two key blocks (128 keys)
// per tile:
//
//     S[128 q x 128 keys]  = Q . K_tile^T      tcgen05.mma, A = Q in smem,        B = K in smem
//     O[128 q x 128 d]    += P . V_tile        tcgen05.mma, A = P (bf16) in TMEM, B = V in smem
//
// A key block that only one of the two lists holds is masked for the other half of the rows
// (its softmax weights are written as zero), so the result is exactly the per-block selection.
// Nearby query blocks of video tokens select largely the same key blocks, which is what makes
// the shared tile pay; which two blocks share an item is chosen per call for large list overlap
// (usv_attn_plan.cu).
//
// Query rows live on TMEM lanes: softmax thread i owns row i, so maxima and sums need no
// cross-thread traffic.  The softmax reference of a row (the value subtracted inside the
// exponential) is fixed at the row maximum over the first key block the row may see and never
// changes, so O needs no rescaling; the exponent range of fp32/bf16 absorbs later, larger
// logits.  Rows whose sum leaves [2^-100, 2^100] are reported in a list and recomputed by the
// exact online-softmax kernel, so the result never depends on that assumption.
//
// One persistent CTA per SM, 24 warps, draws items from a global counter (heads with long lists
// first).  Every role runs straight on from one item into the next, so that the tensor pipe
// only drains at the end of the kernel:
//   warps 0-15   four softmax warpgroups sharing the 128 rows (thread r of every group <-> TMEM
//                lane r <-> query row r).  Group g works on the tiles of running parity g >> 1
//                and there on key block g & 1 of the tile (64 logit columns).
//   warps 16-19  output: thread e <-> query row e reads the finished O row out of TMEM a quarter at
//                a time, hands the accumulator back and stores from registers (to o, or, with the
//                unmerge folded in, to every original token that reads the row back), while the
//                softmax groups are already in the next item.
//   warp 20      scout + K producer: draws the next item, copies its key-block list into a ring
//                slot in shared memory and publishes it, fetches Q and the K tiles (TMA).
//   warp 21      P.V issuer and TMEM owner.
//   warp 22      V producer (TMA).
//   warp 23      S issuer.
// The CTA is launched with 80 registers per thread and the roles re-divide them at their start
// (setmaxnreg): the softmax loop needs more than the launch allows for 768 threads, the others less.
//
// TMEM holds O and THREE S buffers; running tile g uses buffer g mod 3.  The weights P are
// written back, as bf16 pairs, into the columns their logits came from, so a buffer goes
// S(g) -> P(g) -> S(g + 3); S(g + 3) is issued once P.V(g) is complete.  Every barrier has
// waiters that see each of its phases (SFULL/PFULL are indexed by g mod 6, the per-item barriers by item mod 4: a waiter that
// skipped a phase could not tell it from the one two before).  All waits are bounded; a wait
// that gives up sets the device status word and every role leaves its loop.
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
constexpr int SBUF = 3;                         // S/P buffers in TMEM
constexpr int NSLOT = 4;                        // item ring
constexpr int LCAP = 512;                       // list entries a ring slot holds (longer lists are read from global memory)
constexpr int MAX_NB = 4096;                    // key blocks per sequence this kernel covers
constexpr uint32_t TILE_BYTES = KT * D * 2;     // 32 KB: [d-half][128 keys][128 B]
constexpr uint32_t SM_Q = 0;                    // the item's 128 query rows, same layout as a K tile
constexpr uint32_t SM_K = SM_Q + TILE_BYTES;
constexpr uint32_t SM_V = SM_K + KSTAGES * TILE_BYTES;
constexpr uint32_t SM_BAR = SM_V + VSTAGES * TILE_BYTES;
// barrier slots (8 bytes each)
enum { B_QFULL = 0, B_QFREE, B_KFULL, B_KEMPTY = B_KFULL + KSTAGES, B_VFULL = B_KEMPTY + KSTAGES,
       B_VEMPTY = B_VFULL + VSTAGES, B_SFULL = B_VEMPTY + VSTAGES, B_PFULL = B_SFULL + 2 * SBUF,
       B_OFULL = B_PFULL + 2 * SBUF, B_OFREE, B_SUMS, B_REF = B_SUMS + NSLOT, B_IFULL = B_REF + 2 * NSLOT,
       B_IFREE = B_IFULL + NSLOT, B_COUNT = B_IFREE + NSLOT };
static_assert(B_COUNT <= 48, "barrier area");
constexpr uint32_t SM_MISC = SM_BAR + 8 * 48;            // tmem base, abort flag
constexpr uint32_t SM_FLAG = SM_MISC + 16;               // int[NSLOT][2]: a row of this side left the safe range
constexpr uint32_t SM_REFV = SM_MISC + 64;               // float[NSLOT][128]: minus the softmax reference per row
constexpr uint32_t SM_SUM = SM_REFV + NSLOT * 128 * 4;   // float[NSLOT][NWG][128]: partial row sums
constexpr uint32_t SM_ITEM = SM_SUM + NSLOT * NWG * 128 * 4;   // NSLOT x { int hdr[16]; int list[LCAP]; }
constexpr uint32_t ITEM_BYTES = 64 + LCAP * 4;
constexpr uint32_t SM_TOTAL = SM_ITEM + NSLOT * ITEM_BYTES;
constexpr size_t SMEM_BYTES = SM_TOTAL + 1024;           // + slack for 1024-byte alignment
static_assert(SMEM_BYTES <= 232448, "shared memory budget");
// item header words
enum { I_T = 0, I_NU, I_B, I_H, I_BH, I_IA, I_IB, I_SREFA, I_SREFB, I_LIST_LO, I_LIST_HI };

// TMEM columns: O | S/P buffer 0 | S/P buffer 1 | S/P buffer 2
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t TO = 0, TS = 128;
static_assert(TS + SBUF * 128 <= TMEM_COLS, "TMEM budget");

constexpr int NSOFT = NWG * 128;   // softmax threads
constexpr int NTHREADS = NSOFT + 128 + 128;   // + output warpgroup + service warpgroup
constexpr int W_EPI = NSOFT / 32, W_TMA = W_EPI + 4, W_MMA = W_EPI + 5, W_TMA_V = W_EPI + 6, W_MMA_S = W_EPI + 7;
// Registers per thread after the roles part ways (setmaxnreg, whole warpgroups).  A CTA can only
// redistribute what it was launched with: 24 warps x 80 registers = 1920 per lane, and
// 16 x 96 + 4 x 56 + 4 x 40 = 1920.  (A request beyond the pool would wait forever.)
constexpr int REG_LAUNCH = 80, REG_SOFT = 96, REG_EPI = 56, REG_SERVICE = 40;
static_assert(16 * REG_SOFT + 4 * REG_EPI + 4 * REG_SERVICE <= 24 * REG_LAUNCH, "register pool of the CTA");

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

// nU entries: (key block << 2) | in-A | in-B << 1, ascending (ring slot or global memory)
__device__ __forceinline__ const int* item_list(const int* hdr) {
    return hdr[I_NU] <= LCAP ? hdr + 16
                             : reinterpret_cast<const int*>(((unsigned long long)(unsigned)hdr[I_LIST_HI] << 32) |
                                                            (unsigned)hdr[I_LIST_LO]);
}

__global__ void __launch_bounds__(NTHREADS, 1)
attn_pair_kernel(const AttnArgs a, const __grid_constant__ Maps maps) {
    dep_launch();   // the set-up below touches shared and tensor memory only; dep_wait() follows it
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* sm = smem_raw + (base - raw);
    auto bar = [&](int i) { return base + SM_BAR + 8u * i; };
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(sm + SM_MISC);
    volatile int* s_abort = reinterpret_cast<volatile int*>(sm + SM_MISC + 4);
    int* s_flag = reinterpret_cast<int*>(sm + SM_FLAG);
    float* s_refv = reinterpret_cast<float*>(sm + SM_REFV);
    float* s_sum = reinterpret_cast<float*>(sm + SM_SUM);
    auto hdr_of = [&](int n) { return reinterpret_cast<int*>(sm + SM_ITEM + (n % NSLOT) * ITEM_BYTES); };

    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int NB = a.NB, N = a.N;
    const int NP = (NB + 1) >> 1;                 // query-block pairs per (b, h)
    const int64_t nitems = (int64_t)a.B * a.H * NP;

    // ---- set-up: barriers (one per thread of the first two warps), TMEM
    if (threadIdx.x < B_COUNT) {
        const int i = threadIdx.x;
        uint32_t count = 1;                                      // Q, K/V stages, SFULL, OFULL, IFULL
        if (i >= B_PFULL && i < B_PFULL + 2 * SBUF) count = 8;   // one per warp of a tile's two groups
        if (i == B_OFREE) count = 4;                             // one per output warp
        if (i >= B_SUMS && i < B_SUMS + NSLOT) count = NSOFT / 32;
        if (i >= B_REF && i < B_REF + 2 * NSLOT) count = 2;      // the two warps of the owning group on a side
        if (i >= B_IFREE && i < B_IFREE + NSLOT) count = 4;      // the output warps read a slot last
        mbar_init(bar(i), count);
        if (i == 0) *s_abort = 0;
        if (i < 2 * NSLOT) s_flag[i] = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == W_MMA) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(base + SM_MISC), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_before();
    __syncthreads();
    fence_after();
    dep_wait();
    const uint32_t tmem = *s_tmem;
    // Each role starts by handing registers over (service and output warps) or taking them
    // (softmax warps): setmaxnreg, whole warpgroups.

    if (warp == W_TMA) {
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REG_SERVICE));
        // ===== scout + K producer (whole warp in the loop, one elected lane issues) ==============
        // publish(n): draw work until an item with at least one key block turns up, copy its list
        // into ring slot n and publish it; a pair without any key block gets its defined output
        // (zeros) right here and is not published.  Returns the item's tile count, -1 after
        // publishing the end marker, -2 when a bounded wait gave up.
        auto publish = [&](int n) -> int {
            int* hdr = hdr_of(n);
            if (n >= NSLOT && !mbar_wait(bar(B_IFREE + n % NSLOT), ((n / NSLOT) - 1) & 1, s_abort, a.status, 0x8000))
                return -2;
            for (;;) {
                int wi = 0;
                if (lane == 0) wi = atomicAdd(a.work_counter, 1);
                const int64_t w = __shfl_sync(0xffffffffu, wi, 0);
                if (w >= nitems) {
                    if (lane == 0) hdr[I_T] = -1;
                    __syncwarp();
                    if (lane == 0) mbar_arrive(bar(B_IFULL + n % NSLOT));
                    return -1;
                }
                const int pair = (int)(w % NP);
                const int bh_ord = (int)(w / NP);
                const int b = bh_ord / a.H;
                const int h = a.head_order[bh_ord % a.H];
                const int2 pq = a.pairs[((int64_t)b * a.H + h) * NP + pair];   // similarity-driven pairing
                const int* pl = a.lists + b * a.list_batch + a.list_off[h] +
                                (int64_t)pair * list_stride(a.k_per_head[h], NB);
                const int nU = __ldg(pl);
                if (nU == 0) {
                    // no valid key block at all: defined output (zeros, log-sum-exp 0), as the exact kernel does
                    __nv_bfloat16* O = a.o + b * a.so.sb + h * a.so.sh;
                    for (int idx = lane; idx < 128 * (D / 8); idx += 32) {
                        const int rr = idx / (D / 8), cc = idx % (D / 8);
                        const int Ir = rr < 64 ? pq.x : pq.y;
                        const int grow = Ir * USV_BLOCK + (rr & 63);
                        if (Ir >= 0 && grow < N) {
                            *reinterpret_cast<uint4*>(O + (int64_t)grow * a.so.sn + cc * 8) = make_uint4(0, 0, 0, 0);
                            if (a.y != nullptr) {
                                const int u1 = a.unmerge_off[(int64_t)b * (N + 1) + grow + 1];
                                for (int u = a.unmerge_off[(int64_t)b * (N + 1) + grow]; u < u1; ++u)
                                    *reinterpret_cast<uint4*>(a.y + ((int64_t)b * a.N_full + a.unmerge_idx[(int64_t)b * a.N_full + u]) *
                                                                        ((int64_t)a.H * D) + h * D + cc * 8) = make_uint4(0, 0, 0, 0);
                            }
                            const int64_t grow_bh = ((int64_t)b * a.H + h) * N + grow;
                            if (a.o_f32 != nullptr) {
                                float4* o32 = reinterpret_cast<float4*>(a.o_f32 + grow_bh * D + cc * 8);
                                o32[0] = make_float4(0.f, 0.f, 0.f, 0.f);
                                o32[1] = make_float4(0.f, 0.f, 0.f, 0.f);
                            }
                            if (a.lse != nullptr && cc == 0) a.lse[grow_bh] = 0.f;
                        }
                    }
                    continue;
                }
                int srefA = nU, srefB = nU;   // first union slot that block A / block B may see
                for (int i0 = 0; i0 < nU; i0 += 32) {
                    const int idx = i0 + lane;
                    const int e = idx < nU ? __ldg(pl + 1 + idx) : 0;
                    if (nU <= LCAP && idx < nU) hdr[16 + idx] = e;
                    const unsigned ba = __ballot_sync(0xffffffffu, e & 1), bb = __ballot_sync(0xffffffffu, e & 2);
                    if (srefA == nU && ba) srefA = i0 + __ffs(ba) - 1;
                    if (srefB == nU && bb) srefB = i0 + __ffs(bb) - 1;
                    if (nU > LCAP && srefA < nU && (srefB < nU || pq.y < 0)) break;   // nothing to copy
                }
                if (lane == 0) {
                    hdr[I_T] = (nU + 1) >> 1;   // 128-key tiles
                    hdr[I_NU] = nU;
                    hdr[I_B] = b; hdr[I_H] = h; hdr[I_BH] = bh_ord; hdr[I_IA] = pq.x; hdr[I_IB] = pq.y;
                    hdr[I_SREFA] = srefA; hdr[I_SREFB] = srefB;
                    const unsigned long long lp = reinterpret_cast<unsigned long long>(pl + 1);
                    hdr[I_LIST_LO] = (int)(unsigned)lp; hdr[I_LIST_HI] = (int)(unsigned)(lp >> 32);
                    s_flag[(n % NSLOT) * 2] = 0;
                    s_flag[(n % NSLOT) * 2 + 1] = 0;
                }
                __syncwarp();
                if (lane == 0) mbar_arrive(bar(B_IFULL + n % NSLOT));
                return (nU + 1) >> 1;
            }
        };
        // Q rows of published item m -> the Q buffer, once the last S tile of item m - 1 is done.
        auto load_q = [&](int m) -> bool {
            const int* hdr = hdr_of(m);
            const int b = hdr[I_B], h = hdr[I_H], IA = hdr[I_IA], IB = hdr[I_IB];
            if (m >= 1 && !mbar_wait(bar(B_QFREE), (m - 1) & 1, s_abort, a.status, 0x4000)) return false;
            if (elect_one()) {
                // a block without a partner reads rows past the end (zero fill)
                const int ra = IA * USV_BLOCK, rb = (IB >= 0 ? IB : NB) * USV_BLOCK;
                mbar_expect_tx(bar(B_QFULL), TILE_BYTES);
                tma_load_4d(base + SM_Q, &maps.q, bar(B_QFULL), 0, ra, h, b);
                tma_load_4d(base + SM_Q + 8192, &maps.q, bar(B_QFULL), 0, rb, h, b);
                tma_load_4d(base + SM_Q + 16384, &maps.q, bar(B_QFULL), 64, ra, h, b);
                tma_load_4d(base + SM_Q + 24576, &maps.q, bar(B_QFULL), 64, rb, h, b);
            }
            __syncwarp();
            return true;
        };
        int g = 0;   // running tile counter
        int n = 0;   // running item counter
        int T = publish(0);
        while (T > 0) {
            const int* hdr = hdr_of(n);
            const int nU = hdr[I_NU];
            const int* list = item_list(hdr);
            const int b = hdr[I_B], h = hdr[I_H];
            int Tn = 0;
            bool pub = false, ok = true;
            if (n == 0 && !load_q(0)) break;
            for (int t = 0; t < T; ++t, ++g) {
                // the next item is drawn and published once this one's first tiles are on their
                // way: its global round trips then fall into the wait for the K stages to come back
                if (t == KSTAGES) {
                    Tn = publish(n + 1);
                    pub = true;
                    if (Tn == -2) { ok = false; break; }
                }
                const int s = g % KSTAGES;
                const uint32_t ph = (g / KSTAGES) & 1;
                const int J0 = list[2 * t] >> 2;
                const int J1 = (2 * t + 1 < nU) ? (list[2 * t + 1] >> 2) : J0;  // odd tail: finite filler, masked
                if (!mbar_wait(bar(B_KEMPTY + s), ph ^ 1, s_abort, a.status, 0x1)) { ok = false; break; }
                const uint32_t dst = base + SM_K + s * TILE_BYTES;
                if (elect_one()) {
                    mbar_expect_tx(bar(B_KFULL + s), TILE_BYTES);
                    tma_load_4d(dst, &maps.k, bar(B_KFULL + s), 0, J0 * USV_BLOCK, h, b);
                    tma_load_4d(dst + 8192, &maps.k, bar(B_KFULL + s), 0, J1 * USV_BLOCK, h, b);
                    tma_load_4d(dst + 16384, &maps.k, bar(B_KFULL + s), 64, J0 * USV_BLOCK, h, b);
                    tma_load_4d(dst + 24576, &maps.k, bar(B_KFULL + s), 64, J1 * USV_BLOCK, h, b);
                }
                __syncwarp();
                // This item's Q rows follow its first K tile: the Q buffer comes free one S tile
                // later than that K stage does, and the K tile must not wait for it.
                if (t == 0 && n > 0 && !load_q(n)) { ok = false; break; }
            }
            if (!ok) break;
            if (!pub) {
                Tn = publish(n + 1);
                if (Tn == -2) break;
            }
            ++n;
            T = Tn;
        }
    } else if (warp == W_TMA_V) {
        // ===== V producer ========================================================================
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REG_SERVICE));
        int g = 0;
        for (int n = 0;; ++n) {
            if (!mbar_wait(bar(B_IFULL + n % NSLOT), (n / NSLOT) & 1, s_abort, a.status, 0x10000)) break;
            const int* hdr = hdr_of(n);
            const int T = hdr[I_T];
            if (T < 0) break;
            const int nU = hdr[I_NU];
            const int* list = item_list(hdr);
            const int b = hdr[I_B], h = hdr[I_H];
            bool ok = true;
            for (int t = 0; t < T; ++t, ++g) {
                const int sv = g % VSTAGES;
                const uint32_t phv = (g / VSTAGES) & 1;
                const int J0 = list[2 * t] >> 2;
                const int J1 = (2 * t + 1 < nU) ? (list[2 * t + 1] >> 2) : J0;
                if (!mbar_wait(bar(B_VEMPTY + sv), phv ^ 1, s_abort, a.status, 0x2)) { ok = false; break; }
                const uint32_t dst = base + SM_V + sv * TILE_BYTES;
                if (elect_one()) {
                    mbar_expect_tx(bar(B_VFULL + sv), TILE_BYTES);
                    tma_load_4d(dst, &maps.v, bar(B_VFULL + sv), 0, J0 * USV_BLOCK, h, b);
                    tma_load_4d(dst + 8192, &maps.v, bar(B_VFULL + sv), 0, J1 * USV_BLOCK, h, b);
                    tma_load_4d(dst + 16384, &maps.v, bar(B_VFULL + sv), 64, J0 * USV_BLOCK, h, b);
                    tma_load_4d(dst + 24576, &maps.v, bar(B_VFULL + sv), 64, J1 * USV_BLOCK, h, b);
                }
                __syncwarp();
            }
            if (!ok) break;
        }
    } else if (warp == W_MMA) {
        // ===== P.V issuer (whole warp in the loop, one elected lane issues); TMEM owner ==========
        // Two warps feed the tensor pipe, this one the O += P.V tiles and W_MMA_S the S = Q.K^T tiles:
        // while one of them waits on a barrier or does its bookkeeping, the MMAs of the other keep
        // the pipe busy.  MMAs of different threads are ordered only through barriers: S(g) reuses the
        // TMEM buffer of P(g - 3) and is issued once P.V(g - 3) is COMPLETE (the V stage barrier
        // of that tile says so to the V producer and to the S issuer alike).
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REG_SERVICE));
        constexpr uint32_t IDESC_O = instr_desc(128, D, 0, 1);     // P (TMEM) x V (MN-major)
        const uint64_t vdesc0 = smem_desc(base + SM_V, 16384, 1024);
        int g = 0;                               // running tile
        int p_v = 0, p_buf = 0, p_b6 = 0;        // g % VSTAGES, g % SBUF, g % (2 SBUF)
        uint32_t p_vph = 0, p_ph6 = 0;           // (g / VSTAGES) & 1, (g / (2 SBUF)) & 1
        bool ok = true;
        for (int n = 0; ok; ++n) {
            if (!mbar_wait(bar(B_IFULL + n % NSLOT), (n / NSLOT) & 1, s_abort, a.status, 0x10000)) break;
            const int T = hdr_of(n)[I_T];
            if (T < 0) break;
            for (int t = 0; t < T; ++t, ++g) {
                if (!mbar_wait(bar(B_VFULL + p_v), p_vph, s_abort, a.status, 0x20)) { ok = false; break; }
                if (!mbar_wait(bar(B_PFULL + p_b6), p_ph6, s_abort, a.status, 0x40)) { ok = false; break; }
                // the first P.V of an item overwrites O: the item before must have been read out
                if (t == 0 && n > 0 && !mbar_wait(bar(B_OFREE), (n - 1) & 1, s_abort, a.status, 0x2000)) { ok = false; break; }
                fence_after();
                const uint64_t vdesc = vdesc0 + ((p_v * TILE_BYTES) >> 4);
                const uint32_t pb = tmem + TS + p_buf * 128;   // P: 32 columns at the head of each 64-column half
                if (elect_one()) {
#pragma unroll
                    for (int ks = 0; ks < KT / 16; ++ks)
                        umma_ts(tmem + TO, pb + (ks >> 2) * 64 + (ks & 3) * 8, vdesc + ((ks * 2048) >> 4), IDESC_O,
                                (t > 0 || ks > 0));
                    umma_commit(bar(B_VEMPTY + p_v));      // V stage free; S buffer p_buf free for S(g + 3)
                    if (t == T - 1) umma_commit(bar(B_OFULL));
                }
                __syncwarp();
                if (++p_v == VSTAGES) { p_v = 0; p_vph ^= 1; }
                if (++p_buf == SBUF) p_buf = 0;
                if (++p_b6 == 2 * SBUF) { p_b6 = 0; p_ph6 ^= 1; }
            }
        }
    } else if (warp == W_MMA_S) {
        // ===== S issuer ===========================================================================
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REG_SERVICE));
        static_assert(VSTAGES == SBUF, "the V stage barrier of tile g doubles as the hand-back of S buffer g % SBUF");
        constexpr uint32_t IDESC_S = instr_desc(128, KT, 0, 0);    // Q (K-major) x K (K-major)
        const uint64_t qdesc = smem_desc(base + SM_Q, 16, 1024);        // + byte offset >> 4
        const uint64_t kdesc0 = smem_desc(base + SM_K, 16, 1024);
        int g = 0;
        int s_k = 0, s_buf = 0, s_b6 = 0;      // g % KSTAGES, g % SBUF, g % (2 SBUF)
        uint32_t s_kph = 0, s_bph = 1;         // (g / KSTAGES) & 1; parity of the hand-back of buffer s_buf: ((g / SBUF) & 1) ^ 1
        bool ok = true;
        for (int n = 0; ok; ++n) {
            if (!mbar_wait(bar(B_IFULL + n % NSLOT), (n / NSLOT) & 1, s_abort, a.status, 0x10000)) break;
            const int T = hdr_of(n)[I_T];
            if (T < 0) break;
            if (!mbar_wait(bar(B_QFULL), n & 1, s_abort, a.status, 0x4)) break;
            for (int t = 0; t < T; ++t, ++g) {
                if (!mbar_wait(bar(B_KFULL + s_k), s_kph, s_abort, a.status, 0x8)) { ok = false; break; }
                // buffer s_buf held P(g - 3): P.V(g - 3) must be complete
                if (g >= SBUF && !mbar_wait(bar(B_VEMPTY + s_buf), s_bph, s_abort, a.status, 0x100)) { ok = false; break; }
                fence_after();
                const uint64_t kdesc = kdesc0 + ((s_k * TILE_BYTES) >> 4);
                const uint32_t d_s = tmem + TS + s_buf * 128;
                if (elect_one()) {
#pragma unroll
                    for (int ks = 0; ks < D / 16; ++ks) {
                        const uint32_t off = ((ks >> 2) * 16384 + (ks & 3) * 32) >> 4;
                        umma_ss(d_s, qdesc + off, kdesc + off, IDESC_S, ks > 0);
                    }
                    umma_commit(bar(B_SFULL + s_b6));
                    umma_commit(bar(B_KEMPTY + s_k));             // its K stage may be refilled
                    if (t == T - 1) umma_commit(bar(B_QFREE));    // and, after an item's last tile, the Q buffer
                }
                __syncwarp();
                if (++s_k == KSTAGES) { s_k = 0; s_kph ^= 1; }
                if (++s_buf == SBUF) { s_buf = 0; s_bph ^= 1; }
                if (++s_b6 == 2 * SBUF) s_b6 = 0;
            }
        }
    } else if (warp >= W_EPI && warp < W_TMA) {
        // ===== output warps: thread e <-> TMEM lane e <-> query row e of the item ================
        asm volatile("setmaxnreg.dec.sync.aligned.u32 %0;" ::"n"(REG_EPI));
        const int e = threadIdx.x - NSOFT;
        const int side = e >> 6;                         // 0: block A, 1: block B (uniform per warp)
        const uint32_t lane_base = tmem + ((uint32_t)((warp - W_EPI) * 32) << 16);
        for (int m = 0;; ++m) {
            const int slot = m % NSLOT;
            if (!mbar_wait(bar(B_IFULL + slot), (m / NSLOT) & 1, s_abort, a.status, 0x10000)) break;
            const int* hdr = hdr_of(m);
            if (hdr[I_T] < 0) break;
            const int ib = hdr[I_B], ih = hdr[I_H], ibh = hdr[I_BH], iq = hdr[side ? I_IB : I_IA];
            const bool has_ref = hdr[side ? I_SREFB : I_SREFA] < hdr[I_NU];
            const int row = iq * USV_BLOCK + (e & 63);
            const bool live = iq >= 0 && row < N;
            if (!mbar_wait(bar(B_SUMS + slot), (m / NSLOT) & 1, s_abort, a.status, 0x800)) break;
            const float* sums = s_sum + slot * (NWG * 128);
            float l = 0.f;
#pragma unroll
            for (int q = 0; q < NWG; ++q) l += sums[q * 128 + e];
            const float nref = has_ref ? s_refv[slot * 128 + e] : 0.f;
            const bool in_range = l > 7.9e-31f && l < 1.2e30f;   // ~[2^-100, 2^100]
            if (live && !in_range && a.fallback_list != nullptr && atomicExch(&s_flag[slot * 2 + side], 1) == 0) {
                // first row of this query block to notice: hand the block to the exact kernel
                const int fslot = atomicAdd(a.fallback_count, 1);
                a.fallback_list[fslot] = ibh * NB + iq;
            }
            const float inv = l > 0.f ? 1.0f / l : 0.f;
            if (a.lse != nullptr && live)
                a.lse[((int64_t)ib * a.H + ih) * N + row] = (log2f(l) - nref) * 0.69314718055994531f;
            if (!mbar_wait(bar(B_OFULL), m & 1, s_abort, a.status, 0x200)) break;
            fence_after();
            // The row leaves TMEM a quarter (32 columns) at a time and is stored from registers; the
            // accumulator and the ring slot go back as soon as the last quarter has been read.
            float* o32 = (a.o_f32 != nullptr && live) ? a.o_f32 + (((int64_t)ib * a.H + ih) * N + row) * D : nullptr;
            __nv_bfloat16* O = a.o + ib * a.so.sb + ih * a.so.sh + (int64_t)row * a.so.sn;
            // fused unmerge: the row goes to every original token that reads it back
            int u0 = 0, u1 = 0;
            if (a.y != nullptr && live) {
                u0 = a.unmerge_off[(int64_t)ib * (N + 1) + row];
                u1 = a.unmerge_off[(int64_t)ib * (N + 1) + row + 1];
            }
#pragma unroll 1
            for (int qd = 0; qd < 4; ++qd) {
                uint32_t r0[32];
                tmem_ld32(lane_base + TO + qd * 32, r0);
                tmem_wait_ld();
                if (qd == 3) {
                    fence_before();
                    __syncwarp();
                    if (lane == 0) {
                        mbar_arrive(bar(B_OFREE));
                        mbar_arrive(bar(B_IFREE + slot));
                    }
                }
                if (o32 != nullptr) {
#pragma unroll
                    for (int j = 0; j < 8; ++j)
                        *reinterpret_cast<float4*>(o32 + qd * 32 + j * 4) =
                            make_float4(__uint_as_float(r0[4 * j]) * inv, __uint_as_float(r0[4 * j + 1]) * inv,
                                        __uint_as_float(r0[4 * j + 2]) * inv, __uint_as_float(r0[4 * j + 3]) * inv);
                }
                if (live) {
                    uint4 pk[4];
#pragma unroll
                    for (int i = 0; i < 4; ++i)
                        pk[i] = make_uint4(pack_bf16x2(__uint_as_float(r0[8 * i]) * inv, __uint_as_float(r0[8 * i + 1]) * inv),
                                           pack_bf16x2(__uint_as_float(r0[8 * i + 2]) * inv, __uint_as_float(r0[8 * i + 3]) * inv),
                                           pack_bf16x2(__uint_as_float(r0[8 * i + 4]) * inv, __uint_as_float(r0[8 * i + 5]) * inv),
                                           pack_bf16x2(__uint_as_float(r0[8 * i + 6]) * inv, __uint_as_float(r0[8 * i + 7]) * inv));
                    if (a.y == nullptr) {
#pragma unroll
                        for (int i = 0; i < 4; ++i) *reinterpret_cast<uint4*>(O + qd * 32 + 8 * i) = pk[i];
                    } else {
                        for (int u = u0; u < u1; ++u) {
                            const int tok = a.unmerge_idx[(int64_t)ib * a.N_full + u];
                            __nv_bfloat16* Y = a.y + ((int64_t)ib * a.N_full + tok) * ((int64_t)a.H * D) + ih * D + qd * 32;
#pragma unroll
                            for (int i = 0; i < 4; ++i) *reinterpret_cast<uint4*>(Y + 8 * i) = pk[i];
                        }
                    }
                }
            }
        }
    } else if (warp < W_EPI) {
        // ===== softmax warpgroups ================================================================
        asm volatile("setmaxnreg.inc.sync.aligned.u32 %0;" ::"n"(REG_SOFT));
        const int grp = warp >> 2;                       // tiles of running parity grp >> 1, key block grp & 1
        const int tp = grp >> 1, hb = grp & 1;
        const int r = threadIdx.x & 127;                 // query row within the item, = TMEM lane
        const int side = r >> 6;                         // 0: block A, 1: block B (uniform per warp)
        const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        const float c = a.scale_log2;
        const uint64_t c2 = pack_f32x2(c, c);

        int g = 0;              // running tile counter (first tile of the current item)
        unsigned refph = 0;     // bit s: phase of this side's reference barrier of ring slot s
        bool ok = true;
        for (int n = 0; ok; ++n) {
            if (!mbar_wait(bar(B_IFULL + n % NSLOT), (n / NSLOT) & 1, s_abort, a.status, 0x10000)) { ok = false; break; }
            const int* hdr = hdr_of(n);
            const int T = hdr[I_T];
            if (T < 0) break;
            const int slot_n = n % NSLOT;
            const int nU = hdr[I_NU];
            const int* list = item_list(hdr);
            // sref: first union slot whose key block this row may see (uniform over the query
            // block): the group that owns that slot fixes the row's softmax reference there and
            // publishes it; the other groups pick it up before their first later slot.
            const int sref = hdr[side ? I_SREFB : I_SREFA];
            const uint32_t ref_bar = bar(B_REF + side * NSLOT + slot_n);
            const uint32_t ref_phase = (refph >> slot_n) & 1;
            float* refv = s_refv + slot_n * 128;
            float nref = 0.f;         // minus the softmax reference (base-2, scaled)
            bool have_ref = false;
            uint64_t lr2 = 0;         // two partial sums of the weights this thread produced for its row
            uint64_t nref2 = 0;
            for (int t = (tp - g) & 1; t < T; t += 2) {   // tiles of this item whose running index has parity tp
                const int gt = g + t;                     // running tile index: buffer gt % SBUF, barrier gt % (2 SBUF)
                const int slot = 2 * t + hb;
                const int e = slot < nU ? list[slot] : 0;
                const bool mine = (e >> side) & 1;
                const int nv = N - (e >> 2) * USV_BLOCK;   // keys of the block with index < N
                const int b6 = gt % (2 * SBUF);
                const uint32_t ph6 = (gt / (2 * SBUF)) & 1;
                const uint32_t sbase = lane_base + TS + (gt % SBUF) * 128 + hb * 64;
                if (!mbar_wait(bar(B_SFULL + b6), ph6, s_abort, a.status, 0x80)) { ok = false; break; }
                fence_after();
                if (!have_ref && sref < nU && slot >= sref) {   // (a side without any key block has sref = nU)
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
                        refv[r] = nref;
                        __syncwarp();
                        if (lane == 0) mbar_arrive(ref_bar);
                    } else {
                        if (!mbar_wait(ref_bar, ref_phase, s_abort, a.status, 0x400)) { ok = false; break; }
                        nref = refv[r];
                    }
                    nref2 = pack_f32x2(nref, nref);
                    have_ref = true;
                }
                // The weights (bf16 pairs) go back into the columns their logits came from: P takes
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
                if (lane == 0) mbar_arrive(bar(B_PFULL + b6));
            }
            if (!ok) break;
            if (sref < nU) refph ^= 1u << slot_n;
            float lr_lo, lr_hi;
            unpack_f32x2(lr2, lr_lo, lr_hi);
            s_sum[slot_n * (NWG * 128) + grp * 128 + r] = lr_lo + lr_hi;
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(B_SUMS + slot_n));
            g += T;
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
    if (warp == W_MMA) {
        fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
    }
}

// Fused unmerge: query blocks the exact kernel recomputed sit in o; copy them to their tokens in y.
__global__ void __launch_bounds__(128) scatter_fallback_kernel(const AttnArgs a) {
    dep_sync();
    const int count = *a.fallback_count;
    const int NB = a.NB, N = a.N;
    for (int w = blockIdx.x; w < count; w += gridDim.x) {
        const int id = a.fallback_list[w];
        const int I = id % NB, bh_ord = id / NB;
        const int b = bh_ord / a.H, h = a.head_order[bh_ord % a.H];
        for (int idx = threadIdx.x; idx < USV_BLOCK * (D / 8); idx += 128) {
            const int rr = idx / (D / 8), cc = idx % (D / 8);
            const int row = I * USV_BLOCK + rr;
            if (row >= N) continue;
            const uint4 val = *reinterpret_cast<const uint4*>(a.o + b * a.so.sb + h * a.so.sh + (int64_t)row * a.so.sn + cc * 8);
            const int u0 = a.unmerge_off[(int64_t)b * (N + 1) + row], u1 = a.unmerge_off[(int64_t)b * (N + 1) + row + 1];
            for (int u = u0; u < u1; ++u) {
                const int tok = a.unmerge_idx[(int64_t)b * a.N_full + u];
                *reinterpret_cast<uint4*>(a.y + ((int64_t)b * a.N_full + tok) * ((int64_t)a.H * D) + h * D + cc * 8) = val;
            }
        }
    }
}

}  // namespace pr

int launch_scatter_fallbacks(const AttnArgs& a, int d, cudaStream_t st) {
    (void)d;
    launch_dep(pr::scatter_fallback_kernel, dim3(64), dim3(128), 0, st, a);
    USV_CHECK_LAUNCH("scatter_fallback_kernel");
    return USV_OK;
}

bool attn_pair_supported(const AttnArgs& a, int d) {
    return d == pr::D && a.NB <= pr::MAX_NB && a.work_counter != nullptr;
}

int launch_attn_pair(const AttnArgs& a, int d, cudaStream_t st) {
    pr::Maps maps;
    int rc;
    if ((rc = t5::make_bhnd_map(&maps.q, a.q, a.sq, a.B, a.H, a.N, d, "q")) != USV_OK) return rc;
    if ((rc = t5::make_bhnd_map(&maps.k, a.k, a.sk, a.B, a.H, a.N, d, "k")) != USV_OK) return rc;
    if ((rc = t5::make_bhnd_map(&maps.v, a.v, a.sv, a.B, a.H, a.N, d, "v")) != USV_OK) return rc;
    const int64_t items = (int64_t)a.B * a.H * ((a.NB + 1) / 2);
    if (items > 2000000000LL) return fail(USV_ERR_UNSUPPORTED, "sparse_attn: too many query blocks");
    int dev = 0, sms = 0;
    if (cudaGetDevice(&dev) != cudaSuccess ||
        cudaDeviceGetAttribute(&sms, cudaDevAttrMultiProcessorCount, dev) != cudaSuccess || sms <= 0)
        return fail(USV_ERR_CUDA, "sparse_attn: cannot query the SM count");
    const int grid = (int)(items < sms ? items : sms);   // one persistent CTA per SM
    cudaError_t e = cudaFuncSetAttribute(pr::attn_pair_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize,
                                         (int)pr::SMEM_BYTES);
    if (e != cudaSuccess) return fail(USV_ERR_CUDA, "sparse_attn: smem attribute: %s", cudaGetErrorString(e));
    // The roles redistribute the registers the CTA is launched with; a build whose launch count
    // fell below what they ask for in total would leave the softmax warps waiting for registers
    // that never come.  Refuse to launch such a build.
    cudaFuncAttributes fa;
    e = cudaFuncGetAttributes(&fa, pr::attn_pair_kernel);
    if (e != cudaSuccess) return fail(USV_ERR_CUDA, "sparse_attn: kernel attributes: %s", cudaGetErrorString(e));
    if (fa.numRegs * (pr::NTHREADS / 32) < 16 * pr::REG_SOFT + 4 * pr::REG_EPI + 4 * pr::REG_SERVICE)
        return fail(USV_ERR_UNSUPPORTED, "sparse_attn: kernel built with %d registers per thread, the roles need %d per lane",
                    fa.numRegs, 16 * pr::REG_SOFT + 4 * pr::REG_EPI + 4 * pr::REG_SERVICE);
    launch_dep(pr::attn_pair_kernel, dim3(grid), dim3(pr::NTHREADS), pr::SMEM_BYTES, st, a, maps);
    USV_CHECK_LAUNCH("attn_pair_kernel");
    return USV_OK;
}

}  // namespace usv
