// Bipartite matching of token merge (Sec. 3.3, Eq. 8-9) on the tensor cores: for every source
// token the destination with the largest cosine, ties to the lowest destination.
//
// The cosines decide an integer (the arg-max) that is compared with an fp64 evaluation.  All
// N_src x N_dst cosines are computed ONCE, from fp16 roundings of the fp32 unit descriptors
// (8 tcgen05.mma, M = 128 sources, N = 128 destinations, K = 16, per 128 x 128 tile, fp32
// accumulation), which are not exact but carry a rigorous bound: every component is off by at most
// 2^-11 relative, so a cosine of two unit vectors is off by at most sum|a_i b_i| (2^-10 + 2^-22)
// <= 2^-10, plus ~1e-6 of accumulation: EPS = 1e-3.  The true best destination of a source
// therefore has an approximate cosine within 2 EPS of the approximate row maximum.  Each source keeps
// its largest approximate cosines (eight per half of the destination tiles); if the last kept one lies
// below (max - 2 EPS) the true arg-max is among the others, and they are re-evaluated in fp32 (exactly what an fp32 pass over the whole
// row would have chosen among them: ties to the lowest destination).  A source with a full list of
// destinations inside the window (duplicates, near-duplicates) is handed to a plain fp32 scan of
// all its destinations.  The result is the fp32 arg-max for every source, whatever the data.
//
//   half_kernel         fp32 descriptors -> fp16 rows, sources (by rank) and destinations (by
//                       ordinal) apart, zero-padded to multiples of 128 rows
//   match_tc_kernel     one CTA per 128 sources: their rows sit in TMEM as the A operand, the
//                       destination rows stream through shared memory (TMA, 4 stages); warp 8 =
//                       TMA producer, warps 9-10 = MMA issuers on alternate tiles, warps 0-3 / 4-7 =
//                       two groups of one thread per source row, reading the 128 x 128 tiles of even /
//                       odd index out of TMEM (three accumulator tiles in rotation) and keeping the eight best (value,
//                       destination) inside the window of their running maximum, ascending destinations
//   recheck_kernel      per source: the candidates inside the window in fp32 -> j*, u; sources
//                       with a full window are listed
//   match_exact_kernel  fp32 scan of every destination for the listed sources (normally none)
#include <cuda_fp16.h>

#include "usv_match.cuh"
#include "usv_tcgen05.cuh"

namespace usv {

namespace mt {

using namespace t5;

constexpr int DM = 128;
constexpr int STAGES = 4;
constexpr int NBUF = 3;                                 // accumulator tiles in TMEM: the hand-over of a tile between
                                                        // MMA issuer and epilogue takes longer than its MMAs
constexpr uint32_t STAGE_BYTES = 128 * DM * 2;          // 32 KB: fp16 rows of a tile, [d-half][128 rows][128 B]
constexpr int W_PROD = 8, W_MMA0 = 9;                   // warps 0-7: two epilogue warpgroups
constexpr int NCAND = 8;                                // best approximate cosines kept per source and tile parity
constexpr float EPS = 1.0e-3f;                          // bound on |approximate - exact cosine| (see above)
constexpr uint32_t SM_B = 0;
constexpr uint32_t SM_SCR = SM_B + STAGES * STAGE_BYTES;   // float[32][256]: a chunk of one row per epilogue thread
constexpr uint32_t SM_BAR = SM_SCR + 32 * 256 * 4;
enum { B_AFULL = 0, B_BFULL = 1, B_BEMPTY = B_BFULL + STAGES, B_DFULL = B_BEMPTY + STAGES, B_DFREE = B_DFULL + 2 * NBUF,
       B_COUNT = B_DFREE + 2 * NBUF };
static_assert(B_COUNT <= 32, "barrier area");
constexpr uint32_t SM_MISC = SM_BAR + 8 * 32;
constexpr uint32_t SM_TOTAL = SM_MISC + 64;
constexpr size_t SMEM_BYTES = SM_TOTAL + 1024;
constexpr uint32_t TMEM_COLS = 512;
constexpr uint32_t TA = 0, TD = 128;                    // A rows (fp16) at 0; D buffers at 128, 256 and 384
static_assert(TD + NBUF * 128 <= TMEM_COLS, "TMEM budget");

__global__ void __launch_bounds__(256)
half_kernel(const float* __restrict__ mhat, MatchTcArgs m) {
    dep_sync();
    for (int64_t w = (int64_t)blockIdx.x * 256 + threadIdx.x; w < m.zero_words; w += (int64_t)gridDim.x * 256)
        reinterpret_cast<unsigned int*>(m.exact_count)[w] = 0u;
    // one warp per output row (4 floats per lane)
    const int64_t gw = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    const int64_t rows_a = (int64_t)m.B * m.nA_pad, rows_b = (int64_t)m.B * m.nB_pad;
    if (gw >= rows_a + rows_b) return;
    const bool is_b = gw >= rows_a;
    const int64_t rr = is_b ? gw - rows_a : gw;
    const int pad = is_b ? m.nB_pad : m.nA_pad, cnt = is_b ? m.p.nB : m.nA;
    const int b = (int)(rr / pad), i = (int)(rr % pad);
    float4 v = make_float4(0.f, 0.f, 0.f, 0.f);
    if (i < cnt) {
        const int tok = is_b ? m.p.dst_token(i) : m.src_idx[i];
        v = *reinterpret_cast<const float4*>(mhat + ((int64_t)b * m.N + tok) * DM + lane * 4);
    }
    __half2 h01 = __floats2half2_rn(v.x, v.y), h23 = __floats2half2_rn(v.z, v.w);
    uint2 out;
    out.x = *reinterpret_cast<uint32_t*>(&h01);
    out.y = *reinterpret_cast<uint32_t*>(&h23);
    *reinterpret_cast<uint2*>((is_b ? m.b_h : m.a_h) + rr * DM + lane * 4) = out;
    if (!is_b) {
        // A lower bound on the source's row maximum, known before the big product starts: its exact
        // cosine with the destination of its own partition block, less the error bound.  Video
        // tokens mostly match a neighbour, so the bound is usually close to the maximum and the
        // matcher's window is narrow from the first tile on.  (Any value that cannot exceed the
        // approximate row maximum is a valid floor; a poor one only costs time.)
        float floor_v = -INFINITY;
        if (i < cnt) {
            const int own = m.p.dst_token(m.p.ord(m.src_idx[i]));
            const float4 y = *reinterpret_cast<const float4*>(mhat + ((int64_t)b * m.N + own) * DM + lane * 4);
            float acc = fmaf(v.x, y.x, fmaf(v.y, y.y, fmaf(v.z, y.z, v.w * y.w)));
#pragma unroll
            for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
            floor_v = acc - 2.0f * EPS;   // exact - EPS bounds its approximate value from below; another EPS of slack
        }
        if (lane == 0) m.floor_v[rr] = floor_v;
    }
}

struct Maps {
    CUtensorMap b_h;
};

// maximum of three fp32 values given as bit patterns (one instruction on this architecture)
__device__ __forceinline__ float max3(uint32_t a, uint32_t b, uint32_t c) {
    float d;
    asm("max.f32 %0, %1, %2, %3;" : "=f"(d) : "f"(__uint_as_float(a)), "f"(__uint_as_float(b)), "f"(__uint_as_float(c)));
    return d;
}

__device__ __forceinline__ void tma_load_2d(uint32_t dst, const CUtensorMap* map, uint32_t bar, int c0, int c1) {
    asm volatile(
        "cp.async.bulk.tensor.2d.shared::cluster.global.mbarrier::complete_tx::bytes [%0], [%1, {%3, %4}], [%2];"
        ::"r"(dst), "l"(reinterpret_cast<uint64_t>(map)), "r"(bar), "r"(c0), "r"(c1)
        : "memory");
}

__global__ void __launch_bounds__(352, 1)
match_tc_kernel(const MatchTcArgs m, const __grid_constant__ Maps maps) {
    dep_launch();   // the set-up below touches shared and tensor memory only; dep_wait() follows it
    extern __shared__ unsigned char smem_raw[];
    const uint32_t raw = smem_u32(smem_raw);
    const uint32_t base = (raw + 1023u) & ~1023u;
    unsigned char* sm = smem_raw + (base - raw);
    auto bar = [&](int i) { return base + SM_BAR + 8u * i; };
    volatile uint32_t* s_tmem = reinterpret_cast<volatile uint32_t*>(sm + SM_MISC);
    volatile int* s_abort = reinterpret_cast<volatile int*>(sm + SM_MISC + 4);
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int b = blockIdx.y;
    const int a0 = blockIdx.x * 128;
    const int T = m.nB_pad / 128;   // destination tiles, walked in the same order by every CTA (walking them
                                    // in rotated orders, so that the CTAs ask for different L2 lines, was slower)

    if (threadIdx.x == 0) {
        mbar_init(bar(B_AFULL), 4);
        for (int s = 0; s < STAGES; ++s) {
            mbar_init(bar(B_BFULL + s), 1);
            mbar_init(bar(B_BEMPTY + s), 1);
        }
        // Tile t uses accumulator t mod NBUF but the barriers t mod (2 NBUF): consecutive uses of an
        // accumulator belong to different issuer warps and epilogue groups (t and t + NBUF differ in
        // parity), and a waiter must see every phase of the barrier it waits on.
        for (int s = 0; s < 2 * NBUF; ++s) {
            mbar_init(bar(B_DFULL + s), 1);
            mbar_init(bar(B_DFREE + s), 4);
        }
        *s_abort = 0;
        asm volatile("fence.mbarrier_init.release.cluster;" ::: "memory");
    }
    if (warp == W_MMA0) {
        asm volatile("tcgen05.alloc.cta_group::1.sync.aligned.shared::cta.b32 [%0], %1;"
                     ::"r"(base + SM_MISC), "r"(TMEM_COLS) : "memory");
        asm volatile("tcgen05.relinquish_alloc_permit.cta_group::1.sync.aligned;" ::: "memory");
    }
    fence_before();
    __syncthreads();
    fence_after();
    dep_wait();
    const uint32_t tmem = *s_tmem;

    if (warp == W_PROD) {
        // ===== TMA producer: destination rows =====
        const int row0 = b * m.nB_pad;
        for (int t = 0; t < T; ++t) {
            const int s = t % STAGES;
            const uint32_t ph = (t / STAGES) & 1;
            if (!mbar_wait(bar(B_BEMPTY + s), ph ^ 1, s_abort, m.status, 0x10000)) break;
            const uint32_t dst = base + SM_B + s * STAGE_BYTES;
            if (elect_one()) {
                mbar_expect_tx(bar(B_BFULL + s), STAGE_BYTES);
                tma_load_2d(dst, &maps.b_h, bar(B_BFULL + s), 0, row0 + t * 128);
                tma_load_2d(dst + 16384, &maps.b_h, bar(B_BFULL + s), 64, row0 + t * 128);
            }
            __syncwarp();
        }
    } else if (warp == W_MMA0 || warp == W_MMA0 + 1) {
        // ===== two MMA issuers: warp 5 takes the even tiles, warp 6 the odd ones (each tile has its
        // own B stage and accumulator tile), so that one warp's barrier waits fall under the other's MMAs =====
        constexpr uint32_t IDESC = instr_desc_f16(128, 128, 0, 0);   // fp16 A (TMEM) x fp16 B (K-major) -> fp32
        const uint64_t bdesc0 = smem_desc(base + SM_B, 16, 1024);
        bool ok = mbar_wait(bar(B_AFULL), 0, s_abort, m.status, 0x20000);
        for (int t = warp - W_MMA0; ok && t < T; t += 2) {
            const int s = t % STAGES;
            const uint32_t ph = (t / STAGES) & 1;
            const int buf = t % NBUF;
            if (!mbar_wait_spin(bar(B_BFULL + s), ph, s_abort, m.status, 0x40000)) break;
            if (t >= NBUF && !mbar_wait_spin(bar(B_DFREE + (t - NBUF) % (2 * NBUF)), ((t - NBUF) / (2 * NBUF)) & 1, s_abort, m.status, 0x80000)) break;
            fence_after();
            const uint64_t bd = bdesc0 + ((s * STAGE_BYTES) >> 4);
            const uint32_t d = tmem + TD + buf * 128;
            if (elect_one()) {
#pragma unroll
                for (int ks = 0; ks < DM / 16; ++ks)
                    umma_ts(d, tmem + TA + ks * 8, bd + (((ks >> 2) * 16384 + (ks & 3) * 32) >> 4), IDESC, ks > 0);
                umma_commit(bar(B_BEMPTY + s));
                umma_commit(bar(B_DFULL + t % (2 * NBUF)));
            }
            __syncwarp();
        }
    } else {
        // ===== two warpgroups, one thread per source row in each: group e reads the tiles of parity e
        // (accumulator tile t mod NBUF) and keeps its own candidates; the two lists meet in recheck_kernel =====
        const int eg = warp >> 2;           // 0: even tiles, 1: odd tiles
        const int r = threadIdx.x & 127;    // TMEM lane = source row of the CTA
        const int a = a0 + r;
        const uint32_t lane_base = tmem + ((uint32_t)((warp & 3) * 32) << 16);
        if (eg == 0) {
            const int64_t row = (int64_t)b * m.nA_pad + a;    // padded: always in range
            const uint4* ph = reinterpret_cast<const uint4*>(m.a_h + row * DM);
#pragma unroll
            for (int c4 = 0; c4 < 4; ++c4) {
                uint32_t q[16];
#pragma unroll
                for (int i = 0; i < 4; ++i) {
                    const uint4 v = __ldg(ph + c4 * 4 + i);
                    q[4 * i] = v.x; q[4 * i + 1] = v.y; q[4 * i + 2] = v.z; q[4 * i + 3] = v.w;
                }
                tmem_st16(lane_base + TA + c4 * 16, q);
            }
            tmem_wait_st();
            fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(B_AFULL));
        }
        // The NCAND largest approximate cosines so far (registers), descending; equal values keep
        // the order of their destinations (ascending), so the lowest destination of a tie stands
        // first.  vmax / vlast mirror the first and the last entry.
        float cval[NCAND];
        int cidx[NCAND];
#pragma unroll
        for (int c = 0; c < NCAND; ++c) { cval[c] = -INFINITY; cidx[c] = 0; }
        float vmax = -INFINITY, vlast = -INFINITY;
        const float floor_v = m.floor_v[(int64_t)b * m.nA_pad + a];   // never above the row's approximate maximum
        bool ok = true;
        for (int t = eg; t < T; t += 2) {
            const int buf = t % NBUF;
            if (!mbar_wait_spin(bar(B_DFULL + t % (2 * NBUF)), (t / (2 * NBUF)) & 1, s_abort, m.status, 0x100000)) { ok = false; break; }
            fence_after();
            const int nvalid = m.p.nB - t * 128;   // destinations of this tile that exist
            // the whole 128-column row in one go (four loads in flight, one wait), then the buffer goes back
            uint32_t sr[128];
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) tmem_ld32(lane_base + TD + buf * 128 + ch * 32, sr + ch * 32);
            tmem_wait_ld();
            fence_before();
            __syncwarp();
            if (lane == 0) mbar_arrive(bar(B_DFREE + t % (2 * NBUF)));
            // The four chunk maxima first (three-input maxima on sixteen independent chains), and
            // from them the tile's: most tiles lie below the window of the running maximum and are done
            // here.  (The maximum only grows, so a destination below the window can never matter.)
            float cm[4];
#pragma unroll
            for (int ch = 0; ch < 4; ++ch) {
                if (nvalid < (ch + 1) * 32) {   // only the chunks of the last tile that reach past the end (uniform)
#pragma unroll
                    for (int j = 0; j < 32; ++j)
                        if (ch * 32 + j >= nvalid) sr[ch * 32 + j] = 0xff800000u;   // -inf: a destination that does not exist
                }
                float c0 = max3(sr[ch * 32], sr[ch * 32 + 1], sr[ch * 32 + 2]);
                float c1 = max3(sr[ch * 32 + 3], sr[ch * 32 + 4], sr[ch * 32 + 5]);
                float c2 = max3(sr[ch * 32 + 6], sr[ch * 32 + 7], sr[ch * 32 + 8]);
                float c3 = max3(sr[ch * 32 + 9], sr[ch * 32 + 10], sr[ch * 32 + 11]);
#pragma unroll
                for (int j = 12; j < 28; j += 8) {
                    c0 = max3(__float_as_uint(c0), sr[ch * 32 + j], sr[ch * 32 + j + 1]);
                    c1 = max3(__float_as_uint(c1), sr[ch * 32 + j + 2], sr[ch * 32 + j + 3]);
                    c2 = max3(__float_as_uint(c2), sr[ch * 32 + j + 4], sr[ch * 32 + j + 5]);
                    c3 = max3(__float_as_uint(c3), sr[ch * 32 + j + 6], sr[ch * 32 + j + 7]);
                }
                c0 = max3(__float_as_uint(c0), sr[ch * 32 + 28], sr[ch * 32 + 29]);
                c1 = max3(__float_as_uint(c1), sr[ch * 32 + 30], sr[ch * 32 + 31]);
                cm[ch] = fmaxf(fmaxf(c0, c1), fmaxf(c2, c3));
            }
            const float tm = fmaxf(fmaxf(cm[0], cm[1]), fmaxf(cm[2], cm[3]));
            if (tm >= fmaxf(vmax, floor_v) - 2.0f * EPS && tm > vlast) {
#pragma unroll
                for (int ch = 0; ch < 4; ++ch) {
                    const float thr = fmaxf(vmax, floor_v) - 2.0f * EPS;
                    if (cm[ch] >= thr && cm[ch] > vlast) {
                        // Rare.  The chunk is parked in shared memory and a bit mask marks the elements
                        // inside the window as it stands; only those are read back and inserted (one
                        // short rolled loop: unrolled over the register elements the insertion is
                        // tens of KB of code, and the kernel then waits on instruction fetch).
                        float* scr = reinterpret_cast<float*>(sm + SM_SCR) + (threadIdx.x & 255);
                        uint32_t mask = 0;
#pragma unroll
                        for (int j = 0; j < 32; ++j) {
                            const float v = __uint_as_float(sr[ch * 32 + j]);
                            scr[j * 256] = v;
                            if (v >= thr && v > vlast) mask |= 1u << j;
                        }
#pragma unroll 1
                        while (mask != 0) {
                            const int j = __ffs(mask) - 1;
                            mask &= mask - 1;
                            const float v = scr[j * 256];
                            if (v >= fmaxf(vmax, floor_v) - 2.0f * EPS && v > vlast) {
                                const int idx = t * 128 + ch * 32 + j;
                                // descending cosine, then ascending destination: the entries the
                                // new one beats move down one place, the last one drops out
                                bool placed = false;
#pragma unroll
                                for (int pos = NCAND - 1; pos > 0; --pos) {
                                    const bool up = v > cval[pos - 1] || (v == cval[pos - 1] && idx < cidx[pos - 1]);
                                    if (!placed) {
                                        cval[pos] = up ? cval[pos - 1] : v;
                                        cidx[pos] = up ? cidx[pos - 1] : idx;
                                    }
                                    placed |= !up;
                                }
                                if (!placed) { cval[0] = v; cidx[0] = idx; }
                                vmax = cval[0];
                                vlast = cval[NCAND - 1];
                            }
                        }
                    }
                }
            }
        }
        if (ok && a < m.nA) {
            const int64_t g4 = (((int64_t)b * m.nA + a) * 2 + eg) * NCAND;
#pragma unroll
            for (int c = 0; c < NCAND; ++c) {
                m.cand_v[g4 + c] = cval[c];
                m.cand_i[g4 + c] = cidx[c];
            }
        }
    }

    fence_before();
    __syncthreads();
    if (*s_abort) {
        const unsigned long long t0 = gtime();
        while (gtime() - t0 < 2000000ull) { }
        __syncthreads();
    }
    if (warp == W_MMA0) {
        fence_after();
        asm volatile("tcgen05.dealloc.cta_group::1.sync.aligned.b32 %0, %1;" ::"r"(tmem), "r"(TMEM_COLS) : "memory");
    }
}

// One warp per source: the candidates inside the window (approximate cosine >= max - 2 EPS) are
// re-evaluated in fp32; the largest wins, equal values go to the lowest destination.  A source whose
// last kept candidate is still inside the window may have more destinations in it than were kept: it is
// appended to the list of the exact scan.
__global__ void __launch_bounds__(256)
recheck_kernel(const float* __restrict__ mhat, MatchTcArgs m) {
    dep_sync();
    const int64_t gw = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    const int lane = threadIdx.x & 31;
    if (gw >= (int64_t)m.B * m.nA) return;
    const int b = (int)(gw / m.nA), a = (int)(gw % m.nA);
    // two lists per source (even and odd destination tiles), each complete for its tiles unless its
    // last entry is still inside the window
    float v[2 * NCAND];
    int id[2 * NCAND];
#pragma unroll
    for (int c = 0; c < 2 * NCAND; ++c) {
        v[c] = m.cand_v[gw * 2 * NCAND + c];
        id[c] = m.cand_i[gw * 2 * NCAND + c];
    }
    const float window = fmaxf(v[0], v[NCAND]) - 2.0f * EPS;
    if (v[NCAND - 1] >= window || v[2 * NCAND - 1] >= window) {   // (never true for -inf entries)
        if (lane == 0) m.exact_list[atomicAdd(m.exact_count, 1)] = (int)gw;
        return;
    }
    const float* M = mhat + (int64_t)b * m.N * DM;
    const float4 x = *reinterpret_cast<const float4*>(M + (int64_t)m.src_idx[a] * DM + lane * 4);
    float best = -INFINITY;
    int bj = 0x7fffffff;
#pragma unroll
    for (int c = 0; c < 2 * NCAND; ++c) {
        if ((c % NCAND) == NCAND - 1 || v[c] < window) continue;   // (uniform over the warp)
        const float4 y = *reinterpret_cast<const float4*>(M + (int64_t)m.p.dst_token(id[c]) * DM + lane * 4);
        float acc = fmaf(x.x, y.x, fmaf(x.y, y.y, fmaf(x.z, y.z, x.w * y.w)));
#pragma unroll
        for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
        if (acc > best || (acc == best && id[c] < bj)) { best = acc; bj = id[c]; }
    }
    if (lane == 0) {
        m.jstar_s[gw] = m.p.dst_token(bj);
        m.u_s[gw] = best;
    }
}

// fp32 scan of every destination for the listed sources (normally few or none): the same
// summation order per cosine as recheck_kernel.  Work unit = (listed source, chunk of 256
// destinations); a warp takes four destinations at a time so that their loads overlap; the best
// (cosine, lowest destination) of a unit goes into the source's slot with one 64-bit atomic maximum
// (order-preserving key of the cosine above, complement of the destination below).
constexpr int EX_CHUNK = 256;

__global__ void __launch_bounds__(256)
match_exact_kernel(const float* __restrict__ mhat, MatchTcArgs m) {
    dep_sync();
    __shared__ unsigned long long s_key[8];
    const int count = *m.exact_count;
    const int nchunks = (m.p.nB + EX_CHUNK - 1) / EX_CHUNK;
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    for (int64_t unit = blockIdx.x; unit < (int64_t)count * nchunks; unit += gridDim.x) {
        const int w = (int)(unit / nchunks), c = (int)(unit % nchunks);
        const int gw = m.exact_list[w];
        const int b = gw / m.nA, a = gw % m.nA;
        const float* M = mhat + (int64_t)b * m.N * DM;
        const float4 x = *reinterpret_cast<const float4*>(M + (int64_t)m.src_idx[a] * DM + lane * 4);
        unsigned long long best = 0ull;
        const int j0 = c * EX_CHUNK + warp * 32;
#pragma unroll 1
        for (int q = 0; q < 32; q += 4) {
            float4 y[4];
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int j = j0 + q + e;
                y[e] = j < m.p.nB ? *reinterpret_cast<const float4*>(M + (int64_t)m.p.dst_token(j) * DM + lane * 4)
                                  : make_float4(0.f, 0.f, 0.f, 0.f);
            }
#pragma unroll
            for (int e = 0; e < 4; ++e) {
                const int j = j0 + q + e;
                float acc = fmaf(x.x, y[e].x, fmaf(x.y, y[e].y, fmaf(x.z, y[e].z, x.w * y[e].w)));
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) acc += __shfl_xor_sync(0xffffffffu, acc, o);
                if (j < m.p.nB) {
                    const unsigned long long key = ((unsigned long long)float_key(acc) << 32) | (0xffffffffu - (unsigned)j);
                    best = key > best ? key : best;
                }
            }
        }
        if (lane == 0) s_key[warp] = best;
        __syncthreads();
        if (threadIdx.x == 0) {
            unsigned long long bb = s_key[0];
            for (int q = 1; q < 8; ++q) bb = s_key[q] > bb ? s_key[q] : bb;
            atomicMax(m.exact_best + w, bb);
        }
        __syncthreads();
    }
}

__global__ void __launch_bounds__(256)
match_exact_finish_kernel(MatchTcArgs m) {
    dep_sync();
    const int count = *m.exact_count;
    for (int w = blockIdx.x * 256 + threadIdx.x; w < count; w += gridDim.x * 256) {
        const unsigned long long key = m.exact_best[w];
        const uint32_t fk = (uint32_t)(key >> 32);
        const uint32_t bits = (fk & 0x80000000u) ? (fk & 0x7fffffffu) : ~fk;    // inverse of float_key
        const int j = (int)(0xffffffffu - (uint32_t)key);
        const int gw = m.exact_list[w];
        m.jstar_s[gw] = m.p.dst_token(j);
        m.u_s[gw] = __uint_as_float(bits);
    }
}

static int make_rows_map(CUtensorMap* map, const void* ptr, int64_t rows, const char* name) {
    EncodeTiledFn fn = encode_fn();
    if (fn == nullptr) return fail(USV_ERR_CUDA, "token_merge: cuTensorMapEncodeTiled not available");
    cuuint64_t dims[2] = {(cuuint64_t)DM, (cuuint64_t)rows};
    cuuint64_t strides[1] = {(cuuint64_t)DM * 2};
    cuuint32_t box[2] = {64, 128};
    cuuint32_t estr[2] = {1, 1};
    CUresult r = fn(map, CU_TENSOR_MAP_DATA_TYPE_FLOAT16, 2, const_cast<void*>(ptr), dims, strides, box, estr,
                    CU_TENSOR_MAP_INTERLEAVE_NONE, CU_TENSOR_MAP_SWIZZLE_128B, CU_TENSOR_MAP_L2_PROMOTION_L2_256B,
                    CU_TENSOR_MAP_FLOAT_OOB_FILL_NONE);
    if (r != CUDA_SUCCESS) return fail(USV_ERR_CUDA, "token_merge: cuTensorMapEncodeTiled(%s) failed with %d", name, (int)r);
    return USV_OK;
}

}  // namespace mt

static inline int pad128(int n) { return (n + 127) / 128 * 128; }

// Layout of the scratch: fp16 rows of sources and destinations (each side padded to 128 rows),
// the candidates (value, destination) per source and tile parity, the list of the exact scan, its counter and results, the floors.
static size_t rows_bytes(int B, int N) { return align_up((size_t)B * ((size_t)N + 256) * mt::DM * sizeof(uint16_t), 256); }
static size_t cand_bytes(int B, int N) { return align_up((size_t)B * N * 2 * mt::NCAND * sizeof(float), 256); }

static size_t list_bytes(int B, int N) { return align_up((size_t)B * N * sizeof(int), 256); }

size_t match_tc_bytes(int B, int N) {
    // rows | candidate values | candidate destinations | exact-scan list | its counter | its results | floors
    return rows_bytes(B, N) + 2 * cand_bytes(B, N) + list_bytes(B, N) + 256 + 2 * list_bytes(B, N) +
           align_up((size_t)B * ((size_t)N + 128) * sizeof(float), 256);
}

int launch_match_tc(const float* mhat, const Part& p, int B, int N, int nA, const int32_t* src_idx,
                    int32_t* jstar_s, float* u_s, void* mem, unsigned int* status, cudaStream_t st) {
    MatchTcArgs m;
    m.p = p; m.B = B; m.N = N; m.nA = nA;
    m.nA_pad = pad128(nA); m.nB_pad = pad128(p.nB);
    m.src_idx = src_idx; m.jstar_s = jstar_s; m.u_s = u_s; m.status = status;
    char* base = static_cast<char*>(mem);
    m.a_h = reinterpret_cast<uint16_t*>(base);
    m.b_h = m.a_h + (size_t)B * m.nA_pad * mt::DM;
    m.cand_v = reinterpret_cast<float*>(base + rows_bytes(B, N));
    m.cand_i = reinterpret_cast<int*>(base + rows_bytes(B, N) + cand_bytes(B, N));
    m.exact_list = reinterpret_cast<int*>(base + rows_bytes(B, N) + 2 * cand_bytes(B, N));
    char* after_list = base + rows_bytes(B, N) + 2 * cand_bytes(B, N) + list_bytes(B, N);
    m.exact_count = reinterpret_cast<int*>(after_list);
    m.exact_best = reinterpret_cast<unsigned long long*>(after_list + 256);
    m.floor_v = reinterpret_cast<float*>(after_list + 256 + 2 * list_bytes(B, N));
    // counter and result slots of the exact scan start at zero: they are adjacent, and half_kernel
    // clears them (a memset between two kernels costs them their overlapped launch)
    m.zero_words = (int)((256 + 2 * list_bytes(B, N)) / 4);
    cudaError_t e;
    const int64_t rows = (int64_t)B * (m.nA_pad + m.nB_pad);
    launch_dep(mt::half_kernel, dim3((unsigned)((rows + 7) / 8)), dim3(256), 0, st, mhat, m);
    USV_CHECK_LAUNCH("half_kernel");
    mt::Maps maps;
    int rc;
    if ((rc = mt::make_rows_map(&maps.b_h, m.b_h, (int64_t)B * m.nB_pad, "b_h")) != USV_OK) return rc;
    e = cudaFuncSetAttribute(mt::match_tc_kernel, cudaFuncAttributeMaxDynamicSharedMemorySize, (int)mt::SMEM_BYTES);
    if (e != cudaSuccess) return fail(USV_ERR_CUDA, "token_merge: smem attribute: %s", cudaGetErrorString(e));
    dim3 grid(m.nA_pad / 128, B);
    launch_dep(mt::match_tc_kernel, dim3(grid), dim3(352), mt::SMEM_BYTES, st, m, maps);
    USV_CHECK_LAUNCH("match_tc_kernel");
    const int64_t srcs = (int64_t)B * nA;
    launch_dep(mt::recheck_kernel, dim3((unsigned)((srcs + 7) / 8)), dim3(256), 0, st, mhat, m);
    USV_CHECK_LAUNCH("recheck_kernel");
    launch_dep(mt::match_exact_kernel, dim3(1184), dim3(256), 0, st, mhat, m);
    USV_CHECK_LAUNCH("match_exact_kernel");
    launch_dep(mt::match_exact_finish_kernel, dim3(8), dim3(256), 0, st, m);
    USV_CHECK_LAUNCH("match_exact_finish_kernel");
    return USV_OK;
}

}  // namespace usv
