// Token merge / unmerge (Sec. 3.3 of the USV paper).
//
//   desc_kernel        Eq. 7-8   head-averaged, unit-normalised key descriptors (HBM stream)
//   src_list_kernel    Eq. 6     ascending list of source tokens of the bipartite partition
//   match_kernel       Eq. 8-9   cosine of every source against every destination of its batch
//                                element with a fused row arg-max (fp32 CUDA cores; the result
//                                decides an integer that is compared with an fp64 evaluation)
//   plan_select_kernel Eq. 10         radix-select of the r-th most confident source
//   plan_assign_kernel Eq. 11, 14     ordered compaction, dst_of / pos
//   csr_* kernels      Eq. 12    sources grouped by destination
//   merge_kernel       Eq. 13-14 warp-per-row gather + mean, 16-byte accesses
//   unmerge_kernel     Eq. 15    warp-per-row gather copy, 16-byte accesses
#include <math.h>

#include "usv_match.cuh"

namespace usv {

// ---------------------------------------------------------------------------- descriptors
// One warp per token.  DM/8 lanes cover one head's row with 16-byte loads; 32/(DM/8) heads are
// read in parallel and combined with shuffles.
template <int DM>
__global__ void __launch_bounds__(256) desc_kernel(const __nv_bfloat16* __restrict__ metric,
                                                   float* __restrict__ mhat, int64_t tokens,
                                                   int Hm) {
    dep_sync();
    constexpr int LPH = DM / 8;    // lanes per head row
    constexpr int HPW = 32 / LPH;  // heads handled at once
    const int64_t tok = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (tok >= tokens) return;
    const int lane = threadIdx.x & 31;
    const int chunk = lane % LPH, hsub = lane / LPH;
    const __nv_bfloat16* src = metric + tok * Hm * DM + chunk * 8;
    float acc[8] = {0, 0, 0, 0, 0, 0, 0, 0};
    for (int h = hsub; h < Hm; h += HPW) {
        float f[8];
        bf16x8_to_float(__ldg(reinterpret_cast<const uint4*>(src + (int64_t)h * DM)), f);
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] += f[e];
    }
#pragma unroll
    for (int o = LPH; o < 32; o <<= 1)
#pragma unroll
        for (int e = 0; e < 8; ++e) acc[e] += __shfl_xor_sync(0xffffffffu, acc[e], o);
    float n2 = 0.f;
    const float invH = 1.0f / (float)Hm;
#pragma unroll
    for (int e = 0; e < 8; ++e) {
        acc[e] *= invH;
        n2 = fmaf(acc[e], acc[e], n2);
    }
#pragma unroll
    for (int o = 1; o < LPH; o <<= 1) n2 += __shfl_xor_sync(0xffffffffu, n2, o);
    const float inv = 1.0f / fmaxf(sqrtf(n2), 1e-12f);
    if (hsub == 0) {
        float* dst = mhat + tok * DM + chunk * 8;
        *reinterpret_cast<float4*>(dst) = make_float4(acc[0] * inv, acc[1] * inv, acc[2] * inv, acc[3] * inv);
        *reinterpret_cast<float4*>(dst + 4) = make_float4(acc[4] * inv, acc[5] * inv, acc[6] * inv, acc[7] * inv);
    }
}

// ---------------------------------------------------------------------------- block scan (1024)
__device__ __forceinline__ int block_scan_1024(int v, int* scratch, int* total) {
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int incl = warp_incl_scan(v);
    if (lane == 31) scratch[warp] = incl;
    __syncthreads();
    if (warp == 0) {
        const int w = scratch[lane];
        const int wi = warp_incl_scan(w);
        scratch[lane] = wi - w;
        if (lane == 31) scratch[32] = wi;
    }
    __syncthreads();
    const int res = scratch[warp] + incl - v;
    *total = scratch[32];
    __syncthreads();
    return res;
}

// Ascending list of the source tokens (same for every batch element): the rank of a source is
// its token index minus the number of destinations before it, which the partition gives in
// closed form, so every token is handled independently.
__global__ void __launch_bounds__(256) src_list_kernel(Part p, int N, int32_t* __restrict__ src_idx) {
    dep_sync();
    const int n = blockIdx.x * 256 + threadIdx.x;
    if (n >= N || p.is_dst(n)) return;
    const int x = n % p.W, y = (n / p.W) % p.Hh, t = n / (p.W * p.Hh);
    int before = ((t + p.st - 1) / p.st) * p.nHy * p.nWx;      // whole destination frames before t
    if (t % p.st == 0) {
        before += ((y + p.sh - 1) / p.sh) * p.nWx;              // whole destination rows before y
        if (y % p.sh == 0) before += (x + p.sw - 1) / p.sw;     // destinations before x in this row
    }
    src_idx[n - before] = n;
}

// ---------------------------------------------------------------------------- matching
// CTA: 256 threads, 64 sources x (all destinations in tiles of 64).  The 64 source descriptors
// stay in shared memory for the whole sweep; destination tiles stream through in chunks of 32
// features.  Each thread keeps the running best of its 4 rows over its 4 columns per tile;
// columns are visited in ascending destination order and replaced only on strict improvement, so
// equal cosines resolve to the lowest destination.
template <int DM>
__global__ void __launch_bounds__(256) match_kernel(const float* __restrict__ mhat, Part p, int N,
                                                    int nA, const int32_t* __restrict__ src_idx,
                                                    int32_t* __restrict__ jstar_s,
                                                    float* __restrict__ u_s) {
    dep_sync();
    constexpr int TK = 32;
    __shared__ __align__(16) float As[DM][64 + 4];
    __shared__ __align__(16) float Bs[TK][64 + 4];
    const int b = blockIdx.y;
    const int a0 = blockIdx.x * 64;
    const float* M = mhat + (int64_t)b * N * DM;
    const int tx = threadIdx.x % 16, ty = threadIdx.x / 16;

    for (int idx = threadIdx.x; idx < 64 * (DM / 4); idx += 256) {
        const int r = idx / (DM / 4), c4 = idx % (DM / 4);
        float4 v = make_float4(0, 0, 0, 0);
        if (a0 + r < nA) v = *reinterpret_cast<const float4*>(M + (int64_t)src_idx[a0 + r] * DM + c4 * 4);
        As[c4 * 4 + 0][r] = v.x; As[c4 * 4 + 1][r] = v.y;
        As[c4 * 4 + 2][r] = v.z; As[c4 * 4 + 3][r] = v.w;
    }
    float best[4] = {-INFINITY, -INFINITY, -INFINITY, -INFINITY};
    int besti[4] = {0x7fffffff, 0x7fffffff, 0x7fffffff, 0x7fffffff};
    __syncthreads();

    for (int j0 = 0; j0 < p.nB; j0 += 64) {
        float acc[4][4] = {};
        for (int k0 = 0; k0 < DM; k0 += TK) {
#pragma unroll
            for (int t = 0; t < 2; ++t) {
                const int idx = threadIdx.x + t * 256;
                const int r = idx / 8, c4 = idx % 8;
                float4 v = make_float4(0, 0, 0, 0);
                if (j0 + r < p.nB)
                    v = *reinterpret_cast<const float4*>(M + (int64_t)p.dst_token(j0 + r) * DM + k0 + c4 * 4);
                Bs[c4 * 4 + 0][r] = v.x; Bs[c4 * 4 + 1][r] = v.y;
                Bs[c4 * 4 + 2][r] = v.z; Bs[c4 * 4 + 3][r] = v.w;
            }
            __syncthreads();
#pragma unroll
            for (int e = 0; e < TK; ++e) {
                const float4 av = *reinterpret_cast<const float4*>(&As[k0 + e][ty * 4]);
                const float4 bv = *reinterpret_cast<const float4*>(&Bs[e][tx * 4]);
                const float ar[4] = {av.x, av.y, av.z, av.w};
                const float br[4] = {bv.x, bv.y, bv.z, bv.w};
#pragma unroll
                for (int i = 0; i < 4; ++i)
#pragma unroll
                    for (int j = 0; j < 4; ++j) acc[i][j] = fmaf(ar[i], br[j], acc[i][j]);
            }
            __syncthreads();
        }
#pragma unroll
        for (int j = 0; j < 4; ++j) {
            const int o = j0 + tx * 4 + j;
            if (o < p.nB) {
#pragma unroll
                for (int i = 0; i < 4; ++i)
                    if (acc[i][j] > best[i]) {
                        best[i] = acc[i][j];
                        besti[i] = o;
                    }
            }
        }
    }
    // combine the 16 threads (consecutive lanes) that share a row
#pragma unroll
    for (int i = 0; i < 4; ++i) {
#pragma unroll
        for (int o = 1; o < 16; o <<= 1) {
            const float ov = __shfl_xor_sync(0xffffffffu, best[i], o);
            const int oi = __shfl_xor_sync(0xffffffffu, besti[i], o);
            if (ov > best[i] || (ov == best[i] && oi < besti[i])) {
                best[i] = ov;
                besti[i] = oi;
            }
        }
        const int a = a0 + ty * 4 + i;
        if (tx == 0 && a < nA) {
            jstar_s[(int64_t)b * nA + a] = p.dst_token(besti[i]);
            u_s[(int64_t)b * nA + a] = best[i];
        }
    }
}

// ---------------------------------------------------------------------------- plan
// One CTA (1024 threads) per batch element.  Radix-select of the r-th largest u, then an ordered
// pass that marks the merged sources (ties to the lowest source index) and writes dst_of / pos.
// Key T of the r-th most confident source and the number of sources equal to T that still merge
// (Eq. 10 with ties to the lowest index), for 0 < r < nA.  One CTA per batch element.
__global__ void __launch_bounds__(1024) plan_select_kernel(int nA, int r, const float* __restrict__ u_s,
                                                           int2* __restrict__ tsel) {
    dep_sync();
    __shared__ int hist[256];
    __shared__ uint32_t s_prefix;
    __shared__ int s_remaining;
    const int b = blockIdx.x;
    const float* u = u_s + (int64_t)b * nA;
    uint32_t T = 0xffffffffu;  // r == 0: nothing is above or equal (need_eq = 0 below)
    int need_eq = 0;
    if (r > 0) {
        if (threadIdx.x == 0) {
            s_prefix = 0;
            s_remaining = r;
        }
        __syncthreads();
        for (int shift = 24; shift >= 0; shift -= 8) {
            if (threadIdx.x < 256) hist[threadIdx.x] = 0;
            __syncthreads();
            const uint32_t prefix = s_prefix;
            const uint32_t mask = shift == 24 ? 0u : (0xffffffffu << (shift + 8));
            for (int a = threadIdx.x; a < nA; a += 1024) {
                const uint32_t key = float_key(u[a]);
                if ((key & mask) == prefix) atomicAdd(&hist[(key >> shift) & 255], 1);
            }
            __syncthreads();
            if (threadIdx.x < 32) {
                const int lane = threadIdx.x;
                const int remaining = s_remaining;
                int local[8], sum = 0;
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    local[t] = hist[255 - (lane * 8 + t)];
                    sum += local[t];
                }
                const int incl = warp_incl_scan(sum);
                int before = incl - sum;
#pragma unroll
                for (int t = 0; t < 8; ++t) {
                    if (before < remaining && remaining <= before + local[t]) {
                        s_prefix = prefix | ((uint32_t)(255 - (lane * 8 + t)) << shift);
                        s_remaining = remaining - before;
                    }
                    before += local[t];
                }
            }
            __syncthreads();
        }
        T = s_prefix;
        need_eq = s_remaining;
    }

    if (threadIdx.x == 0) tsel[b] = make_int2((int)T, need_eq);
}

// Sum over the CTA of one int per thread (1024 threads); `scratch` holds >= 33 ints.
__device__ __forceinline__ int block_sum_1024(int v, int* scratch) {
    int tot;
    block_scan_1024(v, scratch, &tot);
    return tot;
}

// dst_of / pos of the sources (ordered compaction of the unmerged ones, Eq. 11 and 14) and of the
// destinations.  CTA (c, b) owns the sources [1024 c, 1024 c + 1024) of batch element b; what
// it needs to know of the sources before its own (how many are above T, how many equal T) it
// counts itself, so the CTAs are independent.
__global__ void __launch_bounds__(1024) plan_assign_kernel(Part p, int N, int nA, int r, uint32_t T_imm, int need_imm,
                                                           const int2* __restrict__ tsel,
                                                           const int32_t* __restrict__ src_idx,
                                                           const int32_t* __restrict__ jstar_s,
                                                           const float* __restrict__ u_s,
                                                           int32_t* __restrict__ dst_of,
                                                           int32_t* __restrict__ pos,
                                                           float* __restrict__ u_out,
                                                           int32_t* __restrict__ jstar_out,
                                                           int32_t* __restrict__ cnt) {
    dep_sync();
    __shared__ int scratch[33];
    const int b = blockIdx.y;
    const float* u = u_s + (int64_t)b * nA;
    const int32_t* js = jstar_s + (int64_t)b * nA;
    int32_t* d_of = dst_of + (int64_t)b * N;
    int32_t* ps = pos + (int64_t)b * N;
    const int nU = nA - r;
    const uint32_t T = tsel != nullptr ? (uint32_t)tsel[b].x : T_imm;
    const int need_eq = tsel != nullptr ? tsel[b].y : need_imm;
    const int a0 = blockIdx.x * 1024;
    if (a0 < nA) {
        int gt_b = 0, eq_b = 0;
        if (r > 0 && r < nA) {   // otherwise every source, or none, merges: ranks follow from the index
            for (int a = threadIdx.x; a < a0; a += 1024) {
                const uint32_t key = float_key(u[a]);
                gt_b += key > T ? 1 : 0;
                eq_b += key == T ? 1 : 0;
            }
            gt_b = block_sum_1024(gt_b, scratch);
            eq_b = block_sum_1024(eq_b, scratch);
        } else if (r == nA) {
            gt_b = a0;
        }
        const int un_b = a0 - gt_b - min(eq_b, need_eq);   // unmerged sources before this CTA's
        const int a = a0 + threadIdx.x;
        const bool in = a < nA;
        const float ua = in ? u[a] : 0.f;
        const uint32_t key = in ? float_key(ua) : 0u;
        const int is_gt = (in && r > 0 && key > T) ? 1 : 0;
        const int is_eq = (in && r > 0 && key == T) ? 1 : 0;
        int tot;
        const int eq_rank = eq_b + block_scan_1024(is_eq, scratch, &tot);
        const int merged = is_gt | (is_eq && eq_rank < need_eq);
        const int un = (in && !merged) ? 1 : 0;
        const int un_rank = un_b + block_scan_1024(un, scratch, &tot);
        if (in) {
            const int n = src_idx[a];
            const int j = js[a];
            if (merged) {
                d_of[n] = j;
                ps[n] = nU + p.ord(j);
            } else {
                d_of[n] = -1;
                ps[n] = un_rank;
            }
            if (u_out) u_out[(int64_t)b * N + n] = ua;
            if (jstar_out) jstar_out[(int64_t)b * N + n] = j;
        }
    }
    const int o = blockIdx.x * 1024 + threadIdx.x;
    if (o < p.nB) {
        const int n = p.dst_token(o);
        d_of[n] = -1;
        ps[n] = nU + o;
        cnt[(int64_t)b * p.nB + o] = 0;   // the per-destination counts of the CSR pass that follows start at zero
        if (u_out) u_out[(int64_t)b * N + n] = __int_as_float(0x7fc00000);
        if (jstar_out) jstar_out[(int64_t)b * N + n] = -1;
    }
}

// ---------------------------------------------------------------------------- CSR of M(j)
__global__ void __launch_bounds__(256) csr_count_kernel(Part p, int N, int nU,
                                                        const int32_t* __restrict__ dst_of,
                                                        const int32_t* __restrict__ pos,
                                                        int32_t* __restrict__ cnt,
                                                        int32_t* __restrict__ row_src) {
    dep_sync();
    const int b = blockIdx.y;
    const int n = blockIdx.x * 256 + threadIdx.x;
    if (n >= N) return;
    const int j = dst_of[(int64_t)b * N + n];
    if (j >= 0) atomicAdd(&cnt[(int64_t)b * p.nB + p.ord(j)], 1);
    else if (!p.is_dst(n)) row_src[(int64_t)b * nU + pos[(int64_t)b * N + n]] = n;
}

// exclusive scan of cnt[b,:] -> off[b,0..nB], cursor[b,:] = off[b,:nB].  CTA (c, b) owns the
// destinations [1024 c, 1024 c + 1024) and sums the counts before its own itself.
__global__ void __launch_bounds__(1024) csr_scan_kernel(int nB, const int32_t* __restrict__ cnt,
                                                        int32_t* __restrict__ off,
                                                        int32_t* __restrict__ cursor) {
    dep_sync();
    __shared__ int scratch[33];
    const int b = blockIdx.y;
    const int o0 = blockIdx.x * 1024;
    int before = 0;
    for (int o = threadIdx.x; o < o0; o += 1024) before += cnt[(int64_t)b * nB + o];
    int tot;
    block_scan_1024(before, scratch, &tot);
    const int base = tot;
    const int o = o0 + threadIdx.x;
    const int c = o < nB ? cnt[(int64_t)b * nB + o] : 0;
    const int e = base + block_scan_1024(c, scratch, &tot);
    if (o < nB) {
        off[(int64_t)b * (nB + 1) + o] = e;
        cursor[(int64_t)b * nB + o] = e;
    }
    if (o0 + 1024 >= nB && threadIdx.x == 0) off[(int64_t)b * (nB + 1) + nB] = base + tot;
}

__global__ void __launch_bounds__(256) csr_fill_kernel(Part p, int N, int r,
                                                       const int32_t* __restrict__ dst_of,
                                                       int32_t* __restrict__ cursor,
                                                       int32_t* __restrict__ csr) {
    dep_sync();
    const int b = blockIdx.y;
    const int n = blockIdx.x * 256 + threadIdx.x;
    if (n >= N) return;
    const int j = dst_of[(int64_t)b * N + n];
    if (j >= 0) {
        const int slot = atomicAdd(&cursor[(int64_t)b * p.nB + p.ord(j)], 1);
        csr[(int64_t)b * r + slot] = n;
    }
}

// ---------------------------------------------------------------------------- local matching
// The other reading of Sec. 3.3 (matching kept inside neighbouring 3D blocks): Eq. 8-9 with the
// arg-max over the destinations of the partition blocks within (wt, wh, ww) blocks of the
// source's own block.  One warp per source; the lanes split the descriptor, the candidates are
// visited in ascending destination index and a later one wins only when strictly better.
template <int DM>
__global__ void __launch_bounds__(256) match_local_kernel(const float* __restrict__ mhat, Part p, int N, int nA,
                                                          int wt, int wh, int ww,
                                                          const int32_t* __restrict__ src_idx,
                                                          int32_t* __restrict__ jstar_s, float* __restrict__ u_s) {
    dep_sync();
    constexpr int V = DM / 32;   // floats per lane
    const int a = blockIdx.x * 8 + (threadIdx.x >> 5);
    if (a >= nA) return;
    const int b = blockIdx.y;
    const int lane = threadIdx.x & 31;
    const float* mb = mhat + (int64_t)b * N * DM;
    const int i = src_idx[a];
    const int x = i % p.W, y = (i / p.W) % p.Hh, t = i / (p.W * p.Hh);
    const int bt = t / p.st, by = y / p.sh, bx = x / p.sw;
    const int nBt = p.nB / (p.nHy * p.nWx);
    float mi[V];
#pragma unroll
    for (int e = 0; e < V; ++e) mi[e] = mb[(int64_t)i * DM + lane * V + e];
    float best = -INFINITY;
    int jbest = -1;
    for (int ct = max(bt - wt, 0); ct <= min(bt + wt, nBt - 1); ++ct)
        for (int cy = max(by - wh, 0); cy <= min(by + wh, p.nHy - 1); ++cy)
            for (int cx = max(bx - ww, 0); cx <= min(bx + ww, p.nWx - 1); ++cx) {
                const int j = ((ct * p.st) * p.Hh + cy * p.sh) * p.W + cx * p.sw;
                float c = 0.f;
#pragma unroll
                for (int e = 0; e < V; ++e) c = fmaf(mi[e], mb[(int64_t)j * DM + lane * V + e], c);
#pragma unroll
                for (int o = 16; o > 0; o >>= 1) c += __shfl_xor_sync(0xffffffffu, c, o);
                if (c > best) { best = c; jbest = j; }
            }
    if (lane == 0) {
        jstar_s[(int64_t)b * nA + a] = jbest;
        u_s[(int64_t)b * nA + a] = best;
    }
}

// ---------------------------------------------------------------------------- merge
// One warp per output row.  Rows [0,nU) copy an unmerged source; rows [nU, nU+nB) hold a
// destination averaged with its merged sources, summed in ascending source index.
__global__ void __launch_bounds__(256) merge_kernel(Part p, int N, int C, int nU, int Nm, int r,
                                                    const __nv_bfloat16* __restrict__ x,
                                                    const int32_t* __restrict__ row_src,
                                                    const int32_t* __restrict__ off,
                                                    int32_t* __restrict__ csr,
                                                    __nv_bfloat16* __restrict__ out, int64_t rows) {
    dep_sync();
    const int64_t gw = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (gw >= rows) return;
    const int lane = threadIdx.x & 31;
    const int b = (int)(gw / Nm), row = (int)(gw % Nm);
    const __nv_bfloat16* xb = x + (int64_t)b * N * C;
    uint4* dst = reinterpret_cast<uint4*>(out + ((int64_t)b * Nm + row) * C);
    const int nvec = C / 8;
    if (row < nU) {
        const uint4* src = reinterpret_cast<const uint4*>(xb + (int64_t)row_src[(int64_t)b * nU + row] * C);
        for (int c = lane; c < nvec; c += 32) dst[c] = __ldg(src + c);
        return;
    }
    const int o = row - nU;
    const int j = p.dst_token(o);
    const int beg = off[(int64_t)b * (p.nB + 1) + o], end = off[(int64_t)b * (p.nB + 1) + o + 1];
    const int len = end - beg;
    int32_t* list = csr + (int64_t)b * r + beg;
    const uint4* srcj = reinterpret_cast<const uint4*>(xb + (int64_t)j * C);
    if (len == 0) {
        for (int c = lane; c < nvec; c += 32) dst[c] = __ldg(srcj + c);
        return;
    }
    int myid = 0x7fffffff;
    if (len == 1) {
        myid = list[0];
    } else if (len <= 32) {
        // rank sort in registers: lane s ends up holding the s-th smallest source index
        const int id = lane < len ? list[lane] : 0x7fffffff;
        int rank = 0;
#pragma unroll
        for (int s = 0; s < 32; ++s) {
            const int other = __shfl_sync(0xffffffffu, id, s);
            rank += (other < id) ? 1 : 0;
        }
        // ids are distinct, so ranks of the valid lanes are a permutation of 0..len-1
#pragma unroll
        for (int s = 0; s < 32; ++s) {
            const int oid = __shfl_sync(0xffffffffu, id, s);
            const int orank = __shfl_sync(0xffffffffu, rank, s);
            if (orank == lane && s < len) myid = oid;
        }
    } else {
        // rare long list: in-place selection sort of the segment by this warp
        for (int s = 0; s < len - 1; ++s) {
            int bestv = 0x7fffffff, bestp = -1;
            for (int t = s + lane; t < len; t += 32) {
                const int v = list[t];
                if (v < bestv) { bestv = v; bestp = t; }
            }
#pragma unroll
            for (int w = 16; w > 0; w >>= 1) {
                const int ov = __shfl_xor_sync(0xffffffffu, bestv, w);
                const int op = __shfl_xor_sync(0xffffffffu, bestp, w);
                if (ov < bestv) { bestv = ov; bestp = op; }
            }
            if (lane == 0 && bestp != s) {
                const int tmp = list[s];
                list[s] = bestv;
                list[bestp] = tmp;
            }
            __syncwarp();
        }
    }
    const float inv = 1.0f / (float)(len + 1);
    // G 16-byte chunks per lane at a time: the loads of one row are all in flight together, and
    // rows are added in ascending source index (fp32)
    constexpr int G = 3;
    // The destination row and the first two source rows (most destinations have no more) are
    // requested together, before any of them is used.
    const int i0 = len <= 32 ? __shfl_sync(0xffffffffu, myid, 0) : list[0];
    const int i1 = len < 2 ? 0 : (len <= 32 ? __shfl_sync(0xffffffffu, myid, 1) : list[1]);
    const uint4* src0 = reinterpret_cast<const uint4*>(xb + (int64_t)i0 * C);
    const uint4* src1 = reinterpret_cast<const uint4*>(xb + (int64_t)i1 * C);
    for (int c0 = 0; c0 < nvec; c0 += 32 * G) {
        float acc[G][8];
        uint4 v[G], va[G], vb[G];
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const int c = c0 + g * 32 + lane;
            v[g] = c < nvec ? __ldg(srcj + c) : make_uint4(0, 0, 0, 0);
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const int c = c0 + g * 32 + lane;
            va[g] = c < nvec ? __ldg(src0 + c) : make_uint4(0, 0, 0, 0);
        }
        if (len >= 2) {
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const int c = c0 + g * 32 + lane;
                vb[g] = c < nvec ? __ldg(src1 + c) : make_uint4(0, 0, 0, 0);
            }
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
            bf16x8_to_float(v[g], acc[g]);
            float f[8];
            bf16x8_to_float(va[g], f);
#pragma unroll
            for (int e = 0; e < 8; ++e) acc[g][e] += f[e];
        }
        if (len >= 2) {
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float f[8];
                bf16x8_to_float(vb[g], f);
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[g][e] += f[e];
            }
        }
        for (int s = 2; s < len; ++s) {
            const int i = len <= 32 ? __shfl_sync(0xffffffffu, myid, s) : list[s];
            const uint4* srci = reinterpret_cast<const uint4*>(xb + (int64_t)i * C);
#pragma unroll
            for (int g = 0; g < G; ++g) {
                const int c = c0 + g * 32 + lane;
                v[g] = c < nvec ? __ldg(srci + c) : make_uint4(0, 0, 0, 0);
            }
#pragma unroll
            for (int g = 0; g < G; ++g) {
                float f[8];
                bf16x8_to_float(v[g], f);
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[g][e] += f[e];
            }
        }
#pragma unroll
        for (int g = 0; g < G; ++g) {
            const int c = c0 + g * 32 + lane;
            if (c < nvec) {
#pragma unroll
                for (int e = 0; e < 8; ++e) acc[g][e] *= inv;
                dst[c] = float8_to_bf16x8(acc[g]);
            }
        }
    }
}

// ---------------------------------------------------------------------------- unmerge
__global__ void __launch_bounds__(256) unmerge_kernel(int N, int Nm, int C,
                                                      const __nv_bfloat16* __restrict__ ym,
                                                      const int32_t* __restrict__ pos,
                                                      __nv_bfloat16* __restrict__ y, int64_t rows) {
    dep_sync();
    const int64_t gw = (int64_t)blockIdx.x * 8 + (threadIdx.x >> 5);
    if (gw >= rows) return;
    const int lane = threadIdx.x & 31;
    const int b = (int)(gw / N);
    const int pr = pos[gw];
    const uint4* src = reinterpret_cast<const uint4*>(ym + ((int64_t)b * Nm + pr) * C);
    uint4* dst = reinterpret_cast<uint4*>(y + gw * C);
    const int nvec = C / 8;
    for (int c = lane; c < nvec; c += 32) dst[c] = __ldg(src + c);
}

// ---------------------------------------------------------------------------- unmerge map
// Inverse of pos: for every merged row the original tokens that read it back (counting sort by
// merged row; the order inside a row is irrelevant, every token of a row receives the same values).
__global__ void __launch_bounds__(256) inv_count_kernel(int N, int Nm, const int32_t* __restrict__ pos,
                                                        int32_t* __restrict__ cnt) {
    dep_sync();
    const int b = blockIdx.y;
    const int n = blockIdx.x * 256 + threadIdx.x;
    if (n >= N) return;
    const int m = pos[(int64_t)b * N + n];
    if (m >= 0 && m < Nm) atomicAdd(&cnt[(int64_t)b * Nm + m], 1);
}

__global__ void __launch_bounds__(256) inv_fill_kernel(int N, int Nm, const int32_t* __restrict__ pos,
                                                       int32_t* __restrict__ cursor, int32_t* __restrict__ inv_idx) {
    dep_sync();
    const int b = blockIdx.y;
    const int n = blockIdx.x * 256 + threadIdx.x;
    if (n >= N) return;
    const int m = pos[(int64_t)b * N + n];
    if (m >= 0 && m < Nm) inv_idx[(int64_t)b * N + atomicAdd(&cursor[(int64_t)b * Nm + m], 1)] = n;
}

// ---------------------------------------------------------------------------- host side
struct MergeWs {
    size_t mhat, src_idx, jstar_s, u_s, row_src, cnt, off, cursor, csr, status, tsel, split, total;
};

static MergeWs merge_layout(int B, int N, int dm, int nA, int nB) {
    MergeWs w;
    size_t o = 0;
    auto take = [&](size_t bytes) { size_t at = o; o = align_up(o + bytes, 256); return at; };
    w.status = take(WS_HEADER);                                 // workspace header: word 0 = device status word
    w.mhat = take((size_t)B * N * (dm > 0 ? dm : 1) * sizeof(float));
    w.src_idx = take((size_t)nA * 4);
    w.jstar_s = take((size_t)B * nA * 4);
    w.u_s = take((size_t)B * nA * 4);
    w.row_src = take((size_t)B * nA * 4);
    w.cnt = take((size_t)B * nB * 4);
    w.off = take((size_t)B * (nB + 1) * 4);
    w.cursor = take((size_t)B * nB * 4);
    w.csr = take((size_t)B * nA * 4);
    w.tsel = take((size_t)B * sizeof(int2));                    // selection threshold per batch element
    w.split = take(dm == 128 ? match_tc_bytes(B, N) : 0);       // bf16 hi/lo planes of the tensor-core matcher
    w.total = o;
    return w;
}

}  // namespace usv

extern "C" size_t usv_token_merge_workspace(int B, int N, int C, int Hm, int dm) {
    (void)C; (void)Hm;
    if (B <= 0 || N <= 0) return 0;
    // sized for the worst partition (every token but one is a source / a destination)
    return usv::merge_layout(B, N, dm, N, N).total;
}

// win: NULL = arg-max over every destination of the batch element (Eq. 8-9 as printed); else the
// (wt, wh, ww) block window of the local reading.
static int token_merge_impl(int B, int N, int C, const void* x, int Hm, int dm,
                            const void* metric, int T, int Hh, int W, int st, int sh, int sw,
                            int r, void* x_merged, int32_t* dst_of, int32_t* pos, float* u_out,
                            int32_t* jstar_out, void* ws, size_t ws_bytes, void* stream, const int* win) {
    using namespace usv;
    if (win != nullptr && (win[0] < 0 || win[1] < 0 || win[2] < 0))
        return fail(USV_ERR_INVALID_ARG, "token_merge: window (%d,%d,%d) must not be negative", win[0], win[1], win[2]);
    if (B <= 0 || N <= 0 || C <= 0) return fail(USV_ERR_INVALID_ARG, "token_merge: B,N,C must be positive");
    if (T <= 0 || Hh <= 0 || W <= 0 || (int64_t)T * Hh * W != N)
        return fail(USV_ERR_INVALID_ARG, "token_merge: T*Hh*W = %lld != N = %d", (long long)T * Hh * W, N);
    if (st <= 0 || sh <= 0 || sw <= 0) return fail(USV_ERR_INVALID_ARG, "token_merge: partition sizes must be positive");
    if (C % 8) return fail(USV_ERR_UNSUPPORTED, "token_merge: C=%d not a multiple of 8", C);
    if (x == nullptr || x_merged == nullptr || dst_of == nullptr || pos == nullptr || ws == nullptr)
        return fail(USV_ERR_INVALID_ARG, "token_merge: null pointer");
    if (!aligned16(x) || !aligned16(x_merged) || !aligned16(ws))
        return fail(USV_ERR_UNSUPPORTED, "token_merge: x/x_merged/ws not 16-byte aligned");
    Part p;
    p.T = T; p.Hh = Hh; p.W = W; p.st = st; p.sh = sh; p.sw = sw;
    p.nHy = ceil_div(Hh, sh); p.nWx = ceil_div(W, sw);
    p.nB = ceil_div(T, st) * p.nHy * p.nWx;
    const int nA = N - p.nB;
    if (r < 0 || r > nA) return fail(USV_ERR_INVALID_ARG, "token_merge: r=%d outside [0,%d] (number of sources)", r, nA);
    if (metric != nullptr) {
        if (dm != 64 && dm != 128) return fail(USV_ERR_UNSUPPORTED, "token_merge: dm=%d (need 64 or 128)", dm);
        if (Hm <= 0) return fail(USV_ERR_INVALID_ARG, "token_merge: Hm must be positive");
        if (!aligned16(metric)) return fail(USV_ERR_UNSUPPORTED, "token_merge: metric not 16-byte aligned");
    }
    if ((int64_t)B > 65535) return fail(USV_ERR_UNSUPPORTED, "token_merge: B > 65535");
    if (ws_bytes < usv_token_merge_workspace(B, N, C, Hm, dm))
        return fail(USV_ERR_WORKSPACE, "token_merge: workspace %zu < %zu", ws_bytes,
                    usv_token_merge_workspace(B, N, C, Hm, dm));
    const MergeWs L = merge_layout(B, N, dm, nA, p.nB);
    char* base = static_cast<char*>(ws);
    float* mhat = reinterpret_cast<float*>(base + L.mhat);
    int32_t* src_idx = reinterpret_cast<int32_t*>(base + L.src_idx);
    int32_t* jstar_s = reinterpret_cast<int32_t*>(base + L.jstar_s);
    float* u_s = reinterpret_cast<float*>(base + L.u_s);
    int32_t* row_src = reinterpret_cast<int32_t*>(base + L.row_src);
    int32_t* cnt = reinterpret_cast<int32_t*>(base + L.cnt);
    int32_t* off = reinterpret_cast<int32_t*>(base + L.off);
    int32_t* cursor = reinterpret_cast<int32_t*>(base + L.cursor);
    int32_t* csr = reinterpret_cast<int32_t*>(base + L.csr);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    const int nU = nA - r, Nm = N - r;

    if (metric != nullptr) {
        const int64_t tokens = (int64_t)B * N;
        const unsigned dg = (unsigned)((tokens + 7) / 8);
        if (dm == 128) launch_dep(desc_kernel<128>, dim3(dg), dim3(256), 0, s, static_cast<const __nv_bfloat16*>(metric), mhat, tokens, Hm);
        else launch_dep(desc_kernel<64>, dim3(dg), dim3(256), 0, s, static_cast<const __nv_bfloat16*>(metric), mhat, tokens, Hm);
        USV_CHECK_LAUNCH("desc_kernel");
        if (nA > 0) {
            launch_dep(src_list_kernel, dim3(ceil_div(N, 256)), dim3(256), 0, s, p, N, src_idx);
            USV_CHECK_LAUNCH("src_list_kernel");
            if (win != nullptr) {
                dim3 lg(ceil_div(nA, 8), B);
                if (dm == 128) launch_dep(match_local_kernel<128>, dim3(lg), dim3(256), 0, s, mhat, p, N, nA, win[0], win[1], win[2], src_idx, jstar_s, u_s);
                else launch_dep(match_local_kernel<64>, dim3(lg), dim3(256), 0, s, mhat, p, N, nA, win[0], win[1], win[2], src_idx, jstar_s, u_s);
                USV_CHECK_LAUNCH("match_local_kernel");
            } else if (dm == 128) {
                // tensor cores: split-bf16 cosines (usv_match_tc.cu)
                unsigned int* status = reinterpret_cast<unsigned int*>(base + L.status);
                int rc = launch_match_tc(mhat, p, B, N, nA, src_idx, jstar_s, u_s, base + L.split, status, s);
                if (rc != USV_OK) return rc;
            } else {
                dim3 mg(ceil_div(nA, 64), B);
                launch_dep(match_kernel<64>, dim3(mg), dim3(256), 0, s, mhat, p, N, nA, src_idx, jstar_s, u_s);
                USV_CHECK_LAUNCH("match_kernel");
            }
        }
        const int2* tsel = nullptr;
        if (r > 0 && r < nA) {
            int2* tsel_w = reinterpret_cast<int2*>(base + L.tsel);
            launch_dep(plan_select_kernel, dim3(B), dim3(1024), 0, s, nA, r, u_s, tsel_w);
            USV_CHECK_LAUNCH("plan_select_kernel");
            tsel = tsel_w;
        }
        // r = nA: every key is above 0; r = 0: no key is above or equal to the largest one
        dim3 pg(ceil_div(nA > p.nB ? nA : p.nB, 1024), B);
        launch_dep(plan_assign_kernel, dim3(pg), dim3(1024), 0, s, p, N, nA, r, r == nA ? 0u : 0xffffffffu, 0, tsel, src_idx, jstar_s, u_s,
                                               dst_of, pos, u_out, jstar_out, cnt);
        USV_CHECK_LAUNCH("plan_assign_kernel");
    } else {
        cudaError_t e = cudaMemsetAsync(cnt, 0, (size_t)B * p.nB * 4, s);
        if (e != cudaSuccess) return fail(USV_ERR_CUDA, "token_merge: memset: %s", cudaGetErrorString(e));
    }
    dim3 tg(ceil_div(N, 256), B);
    launch_dep(csr_count_kernel, dim3(tg), dim3(256), 0, s, p, N, nU, dst_of, pos, cnt, row_src);
    USV_CHECK_LAUNCH("csr_count_kernel");
    launch_dep(csr_scan_kernel, dim3(dim3(ceil_div(p.nB, 1024), B)), dim3(1024), 0, s, p.nB, cnt, off, cursor);
    USV_CHECK_LAUNCH("csr_scan_kernel");
    if (r > 0) {
        launch_dep(csr_fill_kernel, dim3(tg), dim3(256), 0, s, p, N, r, dst_of, cursor, csr);
        USV_CHECK_LAUNCH("csr_fill_kernel");
    }
    const int64_t rows = (int64_t)B * Nm;
    launch_dep(merge_kernel, dim3((unsigned)((rows + 7) / 8)), dim3(256), 0, s, 
        p, N, C, nU, Nm, r, static_cast<const __nv_bfloat16*>(x), row_src, off, csr,
        static_cast<__nv_bfloat16*>(x_merged), rows);
    USV_CHECK_LAUNCH("merge_kernel");
    return USV_OK;
}

extern "C" int usv_token_unmerge(int B, int N, int Nm, int C, const void* y_merged,
                                 const int32_t* pos, void* y, void* stream) {
    using namespace usv;
    if (B <= 0 || N <= 0 || Nm <= 0 || C <= 0 || Nm > N)
        return fail(USV_ERR_INVALID_ARG, "token_unmerge: need B,N,Nm,C > 0 and Nm <= N");
    if (C % 8) return fail(USV_ERR_UNSUPPORTED, "token_unmerge: C=%d not a multiple of 8", C);
    if (y_merged == nullptr || pos == nullptr || y == nullptr)
        return fail(USV_ERR_INVALID_ARG, "token_unmerge: null pointer");
    if (!aligned16(y_merged) || !aligned16(y))
        return fail(USV_ERR_UNSUPPORTED, "token_unmerge: y_merged/y not 16-byte aligned");
    const int64_t rows = (int64_t)B * N;
    launch_dep(unmerge_kernel, dim3((unsigned)((rows + 7) / 8)), dim3(256), 0, static_cast<cudaStream_t>(stream), 
        N, Nm, C, static_cast<const __nv_bfloat16*>(y_merged), pos,
        static_cast<__nv_bfloat16*>(y), rows);
    USV_CHECK_LAUNCH("unmerge_kernel");
    return USV_OK;
}

// ---------------------------------------------------------------------------- stored plan
// What merge_kernel needs of a plan, kept by the caller beside dst_of / pos so that applying the
// plan to further tensors is the streaming kernel alone: row_src | off | csr | (cnt, cursor scratch),
// each B * (N + 1) ints.
namespace usv {
static size_t cache_stride(int B, int N) { return align_up((size_t)B * ((size_t)N + 1) * sizeof(int32_t), 256); }

static int fill_part(Part& p, int N, int T, int Hh, int W, int st, int sh, int sw, const char* who) {
    if (T <= 0 || Hh <= 0 || W <= 0 || (int64_t)T * Hh * W != N)
        return fail(USV_ERR_INVALID_ARG, "%s: T*Hh*W = %lld != N = %d", who, (long long)T * Hh * W, N);
    if (st <= 0 || sh <= 0 || sw <= 0) return fail(USV_ERR_INVALID_ARG, "%s: partition sizes must be positive", who);
    p.T = T; p.Hh = Hh; p.W = W; p.st = st; p.sh = sh; p.sw = sw;
    p.nHy = ceil_div(Hh, sh); p.nWx = ceil_div(W, sw);
    p.nB = ceil_div(T, st) * p.nHy * p.nWx;
    return USV_OK;
}
}  // namespace usv

extern "C" size_t usv_merge_plan_cache_bytes(int B, int N) {
    if (B <= 0 || N <= 0) return 0;
    return 5 * usv::cache_stride(B, N);
}

extern "C" int usv_merge_plan_cache(int B, int N, int T, int Hh, int W, int st, int sh, int sw, int r,
                                    const int32_t* dst_of, const int32_t* pos, void* cache, size_t cache_bytes,
                                    void* stream) {
    using namespace usv;
    if (B <= 0 || N <= 0) return fail(USV_ERR_INVALID_ARG, "merge_plan_cache: B,N must be positive");
    if (B > 65535) return fail(USV_ERR_UNSUPPORTED, "merge_plan_cache: B > 65535");
    Part p;
    int rc = fill_part(p, N, T, Hh, W, st, sh, sw, "merge_plan_cache");
    if (rc != USV_OK) return rc;
    const int nA = N - p.nB;
    if (r < 0 || r > nA) return fail(USV_ERR_INVALID_ARG, "merge_plan_cache: r=%d outside [0,%d]", r, nA);
    if (dst_of == nullptr || pos == nullptr || cache == nullptr) return fail(USV_ERR_INVALID_ARG, "merge_plan_cache: null pointer");
    if (!aligned16(cache)) return fail(USV_ERR_UNSUPPORTED, "merge_plan_cache: cache not 16-byte aligned");
    if (cache_bytes < usv_merge_plan_cache_bytes(B, N))
        return fail(USV_ERR_WORKSPACE, "merge_plan_cache: cache %zu < %zu", cache_bytes, usv_merge_plan_cache_bytes(B, N));
    char* base = static_cast<char*>(cache);
    const size_t cs = cache_stride(B, N);
    int32_t* row_src = reinterpret_cast<int32_t*>(base);
    int32_t* off = reinterpret_cast<int32_t*>(base + cs);
    int32_t* csr = reinterpret_cast<int32_t*>(base + 2 * cs);
    int32_t* cnt = reinterpret_cast<int32_t*>(base + 3 * cs);
    int32_t* cursor = reinterpret_cast<int32_t*>(base + 4 * cs);
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(cnt, 0, (size_t)B * p.nB * 4, s);
    if (e != cudaSuccess) return fail(USV_ERR_CUDA, "merge_plan_cache: memset: %s", cudaGetErrorString(e));
    dim3 tg(ceil_div(N, 256), B);
    launch_dep(csr_count_kernel, dim3(tg), dim3(256), 0, s, p, N, nA - r, dst_of, pos, cnt, row_src);
    USV_CHECK_LAUNCH("csr_count_kernel");
    launch_dep(csr_scan_kernel, dim3(dim3(ceil_div(p.nB, 1024), B)), dim3(1024), 0, s, p.nB, cnt, off, cursor);
    USV_CHECK_LAUNCH("csr_scan_kernel");
    if (r > 0) {
        launch_dep(csr_fill_kernel, dim3(tg), dim3(256), 0, s, p, N, r, dst_of, cursor, csr);
        USV_CHECK_LAUNCH("csr_fill_kernel");
    }
    return USV_OK;
}

extern "C" int usv_token_merge_apply(int B, int N, int C, const void* x, int T, int Hh, int W, int st, int sh,
                                     int sw, int r, void* cache, void* x_merged, void* stream) {
    using namespace usv;
    if (B <= 0 || N <= 0 || C <= 0) return fail(USV_ERR_INVALID_ARG, "token_merge_apply: B,N,C must be positive");
    if (C % 8) return fail(USV_ERR_UNSUPPORTED, "token_merge_apply: C=%d not a multiple of 8", C);
    Part p;
    int rc = fill_part(p, N, T, Hh, W, st, sh, sw, "token_merge_apply");
    if (rc != USV_OK) return rc;
    const int nA = N - p.nB;
    if (r < 0 || r > nA) return fail(USV_ERR_INVALID_ARG, "token_merge_apply: r=%d outside [0,%d]", r, nA);
    if (x == nullptr || cache == nullptr || x_merged == nullptr) return fail(USV_ERR_INVALID_ARG, "token_merge_apply: null pointer");
    if (!aligned16(x) || !aligned16(x_merged) || !aligned16(cache))
        return fail(USV_ERR_UNSUPPORTED, "token_merge_apply: x/x_merged/cache not 16-byte aligned");
    char* base = static_cast<char*>(cache);
    const size_t cs = cache_stride(B, N);
    const int Nm = N - r;
    const int64_t rows = (int64_t)B * Nm;
    launch_dep(merge_kernel, dim3((unsigned)((rows + 7) / 8)), dim3(256), 0, static_cast<cudaStream_t>(stream), 
        p, N, C, nA - r, Nm, r, static_cast<const __nv_bfloat16*>(x), reinterpret_cast<const int32_t*>(base),
        reinterpret_cast<const int32_t*>(base + cs), reinterpret_cast<int32_t*>(base + 2 * cs),
        static_cast<__nv_bfloat16*>(x_merged), rows);
    USV_CHECK_LAUNCH("merge_kernel");
    return USV_OK;
}

extern "C" size_t usv_unmerge_map_workspace(int B, int Nm) {
    if (B <= 0 || Nm <= 0) return 0;
    return usv::WS_HEADER + 2 * usv::align_up((size_t)B * Nm * sizeof(int32_t), 256);
}

extern "C" int usv_unmerge_map(int B, int N, int Nm, const int32_t* pos, int32_t* inv_off, int32_t* inv_idx,
                               void* ws, size_t ws_bytes, void* stream) {
    using namespace usv;
    if (B <= 0 || N <= 0 || Nm <= 0 || Nm > N) return fail(USV_ERR_INVALID_ARG, "unmerge_map: need B,N,Nm > 0 and Nm <= N");
    if (pos == nullptr || inv_off == nullptr || inv_idx == nullptr || ws == nullptr)
        return fail(USV_ERR_INVALID_ARG, "unmerge_map: null pointer");
    if (B > 65535) return fail(USV_ERR_UNSUPPORTED, "unmerge_map: B > 65535");
    if (ws_bytes < usv_unmerge_map_workspace(B, Nm))
        return fail(USV_ERR_WORKSPACE, "unmerge_map: workspace %zu < %zu", ws_bytes, usv_unmerge_map_workspace(B, Nm));
    int32_t* cnt = reinterpret_cast<int32_t*>(static_cast<char*>(ws) + WS_HEADER);
    int32_t* cursor = reinterpret_cast<int32_t*>(static_cast<char*>(ws) + WS_HEADER + align_up((size_t)B * Nm * 4, 256));
    cudaStream_t s = static_cast<cudaStream_t>(stream);
    cudaError_t e = cudaMemsetAsync(cnt, 0, (size_t)B * Nm * 4, s);
    if (e != cudaSuccess) return fail(USV_ERR_CUDA, "unmerge_map: memset: %s", cudaGetErrorString(e));
    dim3 tg(ceil_div(N, 256), B);
    launch_dep(inv_count_kernel, dim3(tg), dim3(256), 0, s, N, Nm, pos, cnt);
    USV_CHECK_LAUNCH("inv_count_kernel");
    launch_dep(csr_scan_kernel, dim3(dim3(ceil_div(Nm, 1024), B)), dim3(1024), 0, s, Nm, cnt, inv_off, cursor);
    USV_CHECK_LAUNCH("csr_scan_kernel");
    launch_dep(inv_fill_kernel, dim3(tg), dim3(256), 0, s, N, Nm, pos, cursor, inv_idx);
    USV_CHECK_LAUNCH("inv_fill_kernel");
    return USV_OK;
}

extern "C" int usv_token_merge(int B, int N, int C, const void* x, int Hm, int dm,
                               const void* metric, int T, int Hh, int W, int st, int sh, int sw,
                               int r, void* x_merged, int32_t* dst_of, int32_t* pos, float* u_out,
                               int32_t* jstar_out, void* ws, size_t ws_bytes, void* stream) {
    return token_merge_impl(B, N, C, x, Hm, dm, metric, T, Hh, W, st, sh, sw, r, x_merged, dst_of, pos, u_out,
                            jstar_out, ws, ws_bytes, stream, nullptr);
}

extern "C" int usv_token_merge_local(int B, int N, int C, const void* x, int Hm, int dm,
                                     const void* metric, int T, int Hh, int W, int st, int sh, int sw,
                                     int wt, int wh, int ww, int r, void* x_merged, int32_t* dst_of,
                                     int32_t* pos, float* u_out, int32_t* jstar_out, void* ws,
                                     size_t ws_bytes, void* stream) {
    const int win[3] = {wt, wh, ww};
    return token_merge_impl(B, N, C, x, Hm, dm, metric, T, Hh, W, st, sh, sw, r, x_merged, dst_of, pos, u_out,
                            jstar_out, ws, ws_bytes, stream, win);
}
