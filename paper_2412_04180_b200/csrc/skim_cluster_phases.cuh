// Phases of the row-clustering kernels that run after the row has been sorted: distinct-value
// count, binary64 block prefix sums, the one-warp Lloyd iteration for all widths, the error
// table entry and the optional labels (SKIM Algorithm 3; objective of Section 3.2, diagonal form).
// Shared by the generic kernel (skim_cluster.cu) and the fp16-key kernel (skim_cluster16.cu).
#pragma once

#include "skim_internal.cuh"

namespace skimk {

template <typename KeyT> struct KeyOps;

// Order-preserving image of a binary32 value (the scaled path).
template <> struct KeyOps<uint32_t> {
    static constexpr uint32_t PAD = 0xffffffffu;
    __device__ static __forceinline__ uint32_t from_float(float x)
    {
        uint32_t u = __float_as_uint(x);
        return (u & 0x80000000u) ? ~u : (u | 0x80000000u);
    }
    __device__ static __forceinline__ float to_float(uint32_t k)
    {
        return __uint_as_float((k & 0x80000000u) ? (k & 0x7fffffffu) : ~k);
    }
    // key of the largest representable value <= t
    __device__ static __forceinline__ uint32_t floor_key(float t) { return from_float(t); }
    __device__ static __forceinline__ void load8(const uint32_t *p, float *x)
    {
        const uint4 a = *reinterpret_cast<const uint4 *>(p), b = *reinterpret_cast<const uint4 *>(p + 4);
        x[0] = to_float(a.x); x[1] = to_float(a.y); x[2] = to_float(a.z); x[3] = to_float(a.w);
        x[4] = to_float(b.x); x[5] = to_float(b.y); x[6] = to_float(b.z); x[7] = to_float(b.w);
    }
};

// Order-preserving image of a binary16 bit pattern (no scale installed).
template <> struct KeyOps<uint16_t> {
    static constexpr uint16_t PAD = 0xffffu;
    __device__ static __forceinline__ uint16_t from_half_bits(uint16_t h)
    {
        return (h & 0x8000u) ? (uint16_t)~h : (uint16_t)(h | 0x8000u);
    }
    __device__ static __forceinline__ float to_float(uint16_t k)
    {
        uint16_t h = (k & 0x8000u) ? (uint16_t)(k & 0x7fffu) : (uint16_t)~k;
        return __half2float(__ushort_as_half(h));
    }
    __device__ static __forceinline__ uint16_t floor_key(float t)
    {
        uint16_t h = __half_as_ushort(__float2half_rd(t));
        if (h == 0x8000u) h = 0;
        return from_half_bits(h);
    }
    __device__ static __forceinline__ void load8(const uint16_t *p, float *x)
    {
        const uint4 a = *reinterpret_cast<const uint4 *>(p);
        const uint32_t w[4] = {a.x, a.y, a.z, a.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            x[2 * u] = to_float((uint16_t)(w[u] & 0xffffu));
            x[2 * u + 1] = to_float((uint16_t)(w[u] >> 16));
        }
    }
};

struct ClusterArgs {
    const uint16_t *W;
    const float *G;
    const float *rscale;      // nullptr: no scale installed
    const uint8_t *row_bits;  // nullptr: every width
    int64_t rows;
    int64_t ld;
    int m;                    // cols
    int nb, bmin, sumk;
    int iters;
    int blk_shift;            // log2 of the prefix-sum block length (3 or more)
    float *centroids;
    uint8_t *codes;
    float *err;
    unsigned long long *status;
};

struct D3 {
    double a, b, c;
};

__device__ __forceinline__ D3 shfl_up3(D3 v, int off)
{
    D3 r;
    r.a = __shfl_up_sync(0xffffffffu, v.a, off);
    r.b = __shfl_up_sync(0xffffffffu, v.b, off);
    r.c = __shfl_up_sync(0xffffffffu, v.c, off);
    return r;
}

// Small per-block scratch of the phases below.
struct PhaseSmem {
    double wtot[32 * 3];
    double errs[32];
    float tfs[32];
    float dvals[32];
    int misc[4];   // [0] distinct count, [1] slot counter
};

// Adds the first n (0..8) elements of an aligned 8-element group to P, in index order.
template <typename KeyT>
__device__ __forceinline__ void add_group8(const KeyT *k8, const float *g8, int n, bool want_c, D3 &P)
{
    const float4 ga = *reinterpret_cast<const float4 *>(g8), gb = *reinterpret_cast<const float4 *>(g8 + 4);
    const float gs[8] = {ga.x, ga.y, ga.z, ga.w, gb.x, gb.y, gb.z, gb.w};
    float xs[8];
    KeyOps<KeyT>::load8(k8, xs);
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        if (u < n) {
            const double g = (double)gs[u], x = (double)xs[u];
            const double gx = g * x;
            P.a += g;
            P.b += gx;
            if (want_c) P.c = fma(gx, x, P.c);
        }
    }
}

// Number of distinct keys among skeys[0, m) -> ps.misc[0].  Call with all threads; needs a
// __syncthreads() before misc[0] is read (block_prefix_sums ends with one).
template <typename KeyT, int THREADS>
__device__ __forceinline__ void count_distinct(const KeyT *skeys, int m, PhaseSmem &ps)
{
    int local = 0;
    for (int p = threadIdx.x; p < m; p += THREADS) local += (p == 0 || skeys[p] != skeys[p - 1]) ? 1 : 0;
#pragma unroll
    for (int off = 16; off; off >>= 1) local += __shfl_xor_sync(0xffffffffu, local, off);
    if ((threadIdx.x & 31) == 0 && local) atomicAdd(&ps.misc[0], local);
}

// Exclusive binary64 prefix sums of g, g*x, g*x^2 at the start of every block of 2^blk_shift
// sorted elements: PB[q][b] for q = 0..2, b = 0..nblk (entry nblk holds the totals).
// Every warp scans a contiguous range of blocks; the ranges are then offset by the totals of
// the warps before them.  ps.misc[0..1] must have been zeroed (and synced) before the call.
template <typename KeyT, int THREADS>
__device__ __forceinline__ void block_prefix_sums(const KeyT *skeys, const float *sg, int m, int blk_shift, double *PB,
                                                  PhaseSmem &ps)
{
    constexpr int NW = THREADS / 32;
    const int lane = threadIdx.x & 31, warp = threadIdx.x >> 5;
    const int BLK = 1 << blk_shift;
    const int nblk = (m + BLK - 1) >> blk_shift;
    double *PB0 = PB, *PB1 = PB + (nblk + 1), *PB2 = PB + 2 * (nblk + 1);
    const int bpw = (nblk + NW - 1) / NW;
    const int b0 = min(nblk, warp * bpw), b1 = min(nblk, b0 + bpw);
    D3 carry = {0.0, 0.0, 0.0};
    for (int base = b0; base < b1; base += 32) {
        const int b = base + lane;
        D3 v = {0.0, 0.0, 0.0};
        if (b < b1) {
            const int lo = b << blk_shift;
            const int cnt = min(m - lo, BLK);
            for (int c = 0; c < BLK; c += 8) add_group8<KeyT>(skeys + lo + c, sg + lo + c, min(max(cnt - c, 0), 8), true, v);
        }
        D3 inc = v;
#pragma unroll
        for (int off = 1; off < 32; off <<= 1) {
            const D3 t = shfl_up3(inc, off);
            if (lane >= off) { inc.a += t.a; inc.b += t.b; inc.c += t.c; }
        }
        if (b < b1) {
            PB0[b] = carry.a + (inc.a - v.a);
            PB1[b] = carry.b + (inc.b - v.b);
            PB2[b] = carry.c + (inc.c - v.c);
        }
        carry.a += __shfl_sync(0xffffffffu, inc.a, 31);
        carry.b += __shfl_sync(0xffffffffu, inc.b, 31);
        carry.c += __shfl_sync(0xffffffffu, inc.c, 31);
    }
    if (lane == 0) { ps.wtot[warp * 3 + 0] = carry.a; ps.wtot[warp * 3 + 1] = carry.b; ps.wtot[warp * 3 + 2] = carry.c; }
    __syncthreads();
    D3 before = {0.0, 0.0, 0.0};
    for (int w = 0; w < warp; ++w) {
        before.a += ps.wtot[w * 3 + 0];
        before.b += ps.wtot[w * 3 + 1];
        before.c += ps.wtot[w * 3 + 2];
    }
    if (warp > 0) {
        for (int b = b0 + lane; b < b1; b += 32) { PB0[b] += before.a; PB1[b] += before.b; PB2[b] += before.c; }
    }
    if (warp == NW - 1 && lane == 0) {
        PB0[nblk] = before.a + carry.a;
        PB1[nblk] = before.b + carry.b;
        PB2[nblk] = before.c + carry.c;
    }
    __syncthreads();
}

// Rare path: the row has nd <= 16 distinct values; stores them ascending in ps.dvals.
template <typename KeyT, int THREADS>
__device__ __forceinline__ void collect_distinct(const KeyT *skeys, int m, int nd, PhaseSmem &ps)
{
    for (int p = threadIdx.x; p < m; p += THREADS) {
        if (p == 0 || skeys[p] != skeys[p - 1]) {
            const int slot = atomicAdd(&ps.misc[1], 1);
            if (slot < 16) ps.tfs[slot] = __int_as_float(p);
        }
    }
    __syncthreads();
    if (threadIdx.x < 32) {
        const int lane = threadIdx.x;
        const int p = lane < nd ? __float_as_int(ps.tfs[lane]) : 0x7fffffff;
        int rank = 0;
        for (int u = 0; u < nd; ++u) rank += (__shfl_sync(0xffffffffu, p, u) < p) ? 1 : 0;
        __syncwarp();
        if (lane < nd) ps.dvals[rank] = KeyOps<KeyT>::to_float(skeys[p]);
    }
    __syncthreads();
}

// Number of keys <= kt among the sorted skeys[0, m), searched outward from `guess` (the answer of
// the previous iteration; -1: plain binary search).
template <typename KeyT>
__device__ __forceinline__ int upper_bound_near(const KeyT *skeys, int m, KeyT kt, int guess)
{
    int lo = 0, hi = m;
    if (guess >= 0) {
        const bool at = guess < m && skeys[guess] <= kt;
        const bool below = guess > 0 && skeys[guess - 1] > kt;
        if (at) {
            lo = guess + 1;
            for (int step = 1;; step <<= 1) {
                const int idx = lo + step - 1;
                if (idx >= m) { hi = m; break; }
                if (skeys[idx] <= kt) lo = idx + 1; else { hi = idx; break; }
            }
        } else if (below) {
            hi = guess - 1;
            for (int step = 1;; step <<= 1) {
                const int idx = hi - step;
                if (idx < 0) { lo = 0; break; }
                if (skeys[idx] > kt) hi = idx; else { lo = idx + 1; break; }
            }
        } else {
            return guess;
        }
    }
    while (lo < hi) {
        const int mid = (lo + hi) >> 1;
        if (skeys[mid] <= kt) lo = mid + 1; else hi = mid;
    }
    return lo;
}

// Lloyd iterations and the error table entry, run by ONE warp (all 32 lanes must call).
// Lane L owns centroid L of the row's concatenated centroid record and the boundary above it.
// On return ps.tfs[L] holds that boundary (largest binary32 value still assigned to centroid L).
template <typename KeyT>
__device__ __forceinline__ void lloyd_warp(const KeyT *skeys, const float *sg, const double *PB, int nd,
                                           const ClusterArgs &a, int64_t row, PhaseSmem &ps)
{
    using K = KeyOps<KeyT>;
    const int lane = threadIdx.x & 31;
    const int m = a.m;
    const int BLK = 1 << a.blk_shift;
    const int nblk = (m + BLK - 1) >> a.blk_shift;
    const double *PB0 = PB, *PB1 = PB + (nblk + 1), *PB2 = PB + 2 * (nblk + 1);
    int bi = 0, off = 0;
    while (bi < a.nb && lane >= off + (1 << (a.bmin + bi))) { off += 1 << (a.bmin + bi); ++bi; }
    const bool in_set = lane < a.sumk;
    const int width = a.bmin + bi;
    const int k = 1 << width;
    const int j = lane - off;
    const bool wanted = in_set && (!a.row_bits || a.row_bits[row] == width);
    const bool degenerate = wanted && (nd <= k);      // every value gets its own centroid
    const bool normal = wanted && !degenerate;
    const bool has_boundary = wanted && j < k - 1;
    float c = 0.0f;
    if (degenerate) c = ps.dvals[min(j, nd - 1)];
    if (normal) c = K::to_float(skeys[(int)(((long long)(2 * j + 1) * m) / (2 * k))]);

    int Bprev = -1;
    float tf = __int_as_float(0x7f800000);            // +inf: no boundary above the last centroid
    double err_j = 0.0;
    for (int it = 0;; ++it) {
        const float c_up = __shfl_down_sync(0xffffffffu, c, 1);
        int B = m;
        if (has_boundary) {
            // exact midpoint of two binary32 centroids, rounded down to binary32: x <= midpoint
            // holds for a binary32 x exactly when x <= tf
            tf = __double2float_rd(0.5 * ((double)c + (double)c_up));
            if (tf == 0.0f) tf = 0.0f;
            if (normal) B = upper_bound_near<KeyT>(skeys, m, K::floor_key(tf), Bprev);
        }
        const bool same = __all_sync(0xffffffffu, B == Bprev);
        const bool final = (it >= a.iters) || same;
        Bprev = B;
        D3 P = {0.0, 0.0, 0.0};
        if (normal) {
            const int blk = B >> a.blk_shift;
            const int lo = blk << a.blk_shift;
            P.a = PB0[blk];
            P.b = PB1[blk];
            if (final) P.c = PB2[blk];
            const int cnt = B - lo;
            for (int q = 0; q < cnt; q += 8) add_group8<KeyT>(skeys + lo + q, sg + lo + q, min(cnt - q, 8), final, P);
        }
        D3 Q;
        Q.a = __shfl_up_sync(0xffffffffu, P.a, 1);
        Q.b = __shfl_up_sync(0xffffffffu, P.b, 1);
        Q.c = final ? __shfl_up_sync(0xffffffffu, P.c, 1) : 0.0;
        if (j == 0) { Q.a = 0.0; Q.b = 0.0; Q.c = 0.0; }
        const double S0 = P.a - Q.a, S1 = P.b - Q.b;
        if (final) {
            if (normal) {
                const double cd = (double)c, S2 = P.c - Q.c;
                err_j = fmax(fma(cd, fma(cd, S0, -2.0 * S1), S2), 0.0);
            }
            break;
        }
        if (normal && S0 > 0.0) c = (float)(S1 / S0);
    }
    ps.errs[lane] = err_j;
    ps.tfs[lane] = has_boundary ? tf : __int_as_float(0x7f800000);
    __syncwarp();
    if (wanted) {
        if (a.centroids) a.centroids[row * a.sumk + lane] = c;
        if (j == 0 && a.err) {
            double e = 0.0;
            for (int u = 0; u < k; ++u) e += ps.errs[lane + u];
            if (a.row_bits) a.err[row] = (float)e; else a.err[row * a.nb + bi] = (float)e;
        }
    }
}

// Optional labels of the final assignment, in column order (test/diagnostic output).
template <int THREADS>
__device__ __forceinline__ void write_codes(const ClusterArgs &a, int64_t row, const PhaseSmem &ps)
{
    const int m = a.m;
    const uint16_t *Wr = a.W + row * a.ld;
    int only = -1;
    if (a.row_bits) only = (int)a.row_bits[row] - a.bmin;
    for (int e = threadIdx.x; e < m; e += THREADS) {
        float x = __half2float(__ushort_as_half(Wr[e]));
        if (a.rscale) x = __fmul_rn(x, a.rscale[e]);
        int off = 0;
        for (int bi = 0; bi < a.nb; ++bi) {
            const int k = 1 << (a.bmin + bi);
            if (only < 0 || only == bi) {
                int code = 0;
                for (int u = 0; u < k - 1; ++u) code += (ps.tfs[off + u] < x) ? 1 : 0;
                if (only < 0) a.codes[((int64_t)bi * a.rows + row) * m + e] = (uint8_t)code;
                else a.codes[row * (int64_t)m + e] = (uint8_t)code;
            }
            off += k;
        }
    }
}

}  // namespace skimk

// fp16-key kernel (skim_cluster16.cu).  Returns SKIM_OK after launching, or 1 when the call does
// not meet its requirements (then the generic kernel must be used).
int skim_launch_cluster16(skim_ctx *ctx, const skimk::ClusterArgs &args, int64_t rows);
