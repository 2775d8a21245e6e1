// Device code shared by the row-clustering kernels (SKIM Algorithm 3; objective of Section 3.2,
// diagonal form): order-preserving keys, the phases the sort kernels run once a row is sorted
// (distinct-value count, group index, binary64 block prefix sums, the row record), and the one-warp
// Lloyd iteration with the error table entry and the optional labels that the Lloyd kernel runs on
// a row record.  Used by skim_cluster.cu, skim_cluster16.cu and skim_lloyd.cu.
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
    unsigned char *scratch;   // row records of the current chunk (written by the sort kernel, read by the Lloyd kernel)
    long long rec_stride;     // bytes between row records
    int64_t row0;             // first row of the current chunk
};

// Row record: what the sort kernel leaves in global memory for the Lloyd kernel.  All offsets are
// multiples of 16 bytes; values are binary32 whatever key type sorted the row.
//   hdr     int nd (number of distinct values) at byte 0; double totals[3] (sum g, sum g x,
//           sum g x^2 over the row) at byte 16; float dvals[16] at byte 64
//   groups  one 80-byte record per group of 8 sorted elements: 8 values, 8 importances, and the
//           binary64 exclusive prefix sums of g and g*x at the group's first element: everything
//           a boundary needs in one Lloyd iteration.  The last group is padded with the largest
//           finite value and zero importance.
//   gi      group index: first value of every group, sk_entries(m) floats (padded likewise)
//   p2      binary64 exclusive prefix sums of g*x^2 at every group start (ngrp + 1 entries), read
//           once, for the error
struct RowRecord {
    size_t groups, gi, p2, total;
    size_t gi_bytes, p2_bytes;
    int ngrp;
};
constexpr int SKIM_GROUP_BYTES = 80;

__host__ __device__ inline int sk_entries(int m) { return ((((m + 7) >> 3) + 7) & ~7) + 16; }

__host__ __device__ inline RowRecord row_record(int m)
{
    RowRecord R;
    R.ngrp = (m + 7) >> 3;
    R.gi_bytes = (size_t)sk_entries(m) * 4;
    R.p2_bytes = ((size_t)(R.ngrp + 1) * 8 + 15) & ~(size_t)15;
    size_t off = 128;
    R.groups = off; off += (size_t)R.ngrp * SKIM_GROUP_BYTES;
    R.gi = off; off += R.gi_bytes;
    R.p2 = off; off += R.p2_bytes;
    R.total = (off + 127) & ~(size_t)127;
    return R;
}

// Copies `bytes` (a multiple of 16, both pointers 16-byte aligned) with all threads of the block.
template <int THREADS>
__device__ __forceinline__ void copy16(void *dst, const void *src, size_t bytes)
{
    uint4 *d = reinterpret_cast<uint4 *>(dst);
    const uint4 *s = reinterpret_cast<const uint4 *>(src);
    for (size_t i = threadIdx.x; i < bytes / 16; i += THREADS) d[i] = s[i];
}

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
    float tfs[32];     // scratch of collect_distinct
    float dvals[32];   // the row's distinct values when there are at most 16
    int misc[4];       // [0] distinct count, [1] slot counter
};

// An aligned group of 8 sorted elements (keys and importance) held in registers.
template <typename KeyT> struct Group8;

template <> struct Group8<uint16_t> {
    uint4 kv;
    float4 ga, gb;
    __device__ __forceinline__ void load(const uint16_t *k8, const float *g8)
    {
        kv = *reinterpret_cast<const uint4 *>(k8);
        ga = *reinterpret_cast<const float4 *>(g8);
        gb = *reinterpret_cast<const float4 *>(g8 + 4);
    }
    // Number of keys <= kt.  A word holds two ascending keys (low half first): "high half <= kt"
    // is one 32-bit compare against (kt << 16 | 0xffff), "low half <= kt" one compare of the word
    // shifted left by 16.
    __device__ __forceinline__ int count_le(uint16_t kt) const
    {
        const uint32_t khi = ((uint32_t)kt << 16) | 0xffffu, klo = (uint32_t)kt << 16;
        const uint32_t w[4] = {kv.x, kv.y, kv.z, kv.w};
        int c = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q) c += (w[q] <= khi ? 1 : 0) + ((w[q] << 16) <= klo ? 1 : 0);
        return c;
    }
    __device__ __forceinline__ void values(float *x) const
    {
        const uint32_t w[4] = {kv.x, kv.y, kv.z, kv.w};
#pragma unroll
        for (int u = 0; u < 4; ++u) {
            x[2 * u] = KeyOps<uint16_t>::to_float((uint16_t)(w[u] & 0xffffu));
            x[2 * u + 1] = KeyOps<uint16_t>::to_float((uint16_t)(w[u] >> 16));
        }
    }
};

template <> struct Group8<uint32_t> {
    uint4 ka, kb;
    float4 ga, gb;
    __device__ __forceinline__ void load(const uint32_t *k8, const float *g8)
    {
        ka = *reinterpret_cast<const uint4 *>(k8);
        kb = *reinterpret_cast<const uint4 *>(k8 + 4);
        ga = *reinterpret_cast<const float4 *>(g8);
        gb = *reinterpret_cast<const float4 *>(g8 + 4);
    }
    __device__ __forceinline__ int count_le(uint32_t kt) const
    {
        return (ka.x <= kt ? 1 : 0) + (ka.y <= kt ? 1 : 0) + (ka.z <= kt ? 1 : 0) + (ka.w <= kt ? 1 : 0) +
               (kb.x <= kt ? 1 : 0) + (kb.y <= kt ? 1 : 0) + (kb.z <= kt ? 1 : 0) + (kb.w <= kt ? 1 : 0);
    }
    __device__ __forceinline__ void values(float *x) const
    {
        using K = KeyOps<uint32_t>;
        x[0] = K::to_float(ka.x); x[1] = K::to_float(ka.y); x[2] = K::to_float(ka.z); x[3] = K::to_float(ka.w);
        x[4] = K::to_float(kb.x); x[5] = K::to_float(kb.y); x[6] = K::to_float(kb.z); x[7] = K::to_float(kb.w);
    }
};

// Adds the first n (0..8) elements of a group to P.  The eight terms are summed pairwise (a fixed
// order, short dependency chain) and the group total is added to P.  Elements past n are masked
// before any arithmetic touches them.
template <typename KeyT, bool WANT_C>
__device__ __forceinline__ void add_group(const Group8<KeyT> &grp, int n, D3 &P)
{
    const float gs[8] = {grp.ga.x, grp.ga.y, grp.ga.z, grp.ga.w, grp.gb.x, grp.gb.y, grp.gb.z, grp.gb.w};
    float xs[8];
    grp.values(xs);
    double t0[8], t1[8], t2[8];
#pragma unroll
    for (int u = 0; u < 8; ++u) {
        const bool in = u < n;
        const double g = (double)(in ? gs[u] : 0.0f), x = (double)(in ? xs[u] : 0.0f);
        t0[u] = g;
        t1[u] = g * x;
        if (WANT_C) t2[u] = t1[u] * x;
    }
    P.a += ((t0[0] + t0[1]) + (t0[2] + t0[3])) + ((t0[4] + t0[5]) + (t0[6] + t0[7]));
    P.b += ((t1[0] + t1[1]) + (t1[2] + t1[3])) + ((t1[4] + t1[5]) + (t1[6] + t1[7]));
    if (WANT_C) P.c += ((t2[0] + t2[1]) + (t2[2] + t2[3])) + ((t2[4] + t2[5]) + (t2[6] + t2[7]));
}

template <typename KeyT, bool WANT_C>
__device__ __forceinline__ void add_group8(const KeyT *k8, const float *g8, int n, D3 &P)
{
    Group8<KeyT> grp;
    grp.load(k8, g8);
    add_group<KeyT, WANT_C>(grp, n, P);
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
            for (int c = 0; c < BLK; c += 8) add_group8<KeyT, true>(skeys + lo + c, sg + lo + c, min(max(cnt - c, 0), 8), v);
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

// Writes the row record from the block's shared-memory arrays (sorted keys and importance padded
// to whole groups, block prefix sums).  Call with all threads, after block_prefix_sums (and
// collect_distinct when nd <= 16).
template <typename KeyT, int THREADS>
__device__ __forceinline__ void write_row_record(const ClusterArgs &a, const KeyT *skeys, const float *sg, const double *PB,
                                                 int nd, const float *dvals)
{
    const RowRecord R = row_record(a.m);
    unsigned char *rec = a.scratch + (size_t)blockIdx.x * (size_t)a.rec_stride;
    const int BLK = 1 << a.blk_shift;
    const int nblk = (a.m + BLK - 1) >> a.blk_shift;
    const double *PB0 = PB, *PB1 = PB + (nblk + 1), *PB2 = PB + 2 * (nblk + 1);
    const float INF = 3.402823466e38f;   // padding value: the largest finite binary32 (0 * padding stays 0)
    if (threadIdx.x == 0) {
        *reinterpret_cast<int *>(rec) = nd;
        double *tot = reinterpret_cast<double *>(rec + 16);
        tot[0] = PB0[nblk]; tot[1] = PB1[nblk]; tot[2] = PB2[nblk];
    }
    if (threadIdx.x < 16) reinterpret_cast<float *>(rec + 64)[threadIdx.x] = nd <= 16 ? dvals[threadIdx.x] : 0.0f;
    double *p2 = reinterpret_cast<double *>(rec + R.p2);
    float *gi = reinterpret_cast<float *>(rec + R.gi);
    for (int q = threadIdx.x; q < sk_entries(a.m); q += THREADS) {
        if (q >= R.ngrp) {                      // padding of the group index; totals close the p2 array
            gi[q] = INF;
            if (q == R.ngrp) p2[q] = PB2[nblk];
            continue;
        }
        // prefix sums at the start of group q: the block's entry plus the whole groups before q in it
        const int e = q << 3;
        const int blk = e >> a.blk_shift;
        D3 P = {PB0[blk], PB1[blk], PB2[blk]};
        for (int u = blk << a.blk_shift; u < e; u += 8) add_group8<KeyT, true>(skeys + u, sg + u, 8, P);
        p2[q] = P.c;
        float x[8];
        KeyOps<KeyT>::load8(skeys + e, x);
#pragma unroll
        for (int u = 0; u < 8; ++u) {
            if (e + u >= a.m) x[u] = INF;
        }
        gi[q] = x[0];
        unsigned char *gr = rec + R.groups + (size_t)q * SKIM_GROUP_BYTES;
        float4 *xd = reinterpret_cast<float4 *>(gr);
        xd[0] = make_float4(x[0], x[1], x[2], x[3]);
        xd[1] = make_float4(x[4], x[5], x[6], x[7]);
        const float4 *gsrc = reinterpret_cast<const float4 *>(sg + e);
        xd[2] = gsrc[0];
        xd[3] = gsrc[1];
        *reinterpret_cast<double2 *>(gr + 64) = make_double2(P.a, P.b);
    }
}

}  // namespace skimk

// fp16-key sort kernel (skim_cluster16.cu).  Fills args.blk_shift and args.rec_stride when `launch`
// is false (planning) and launches over `rows` rows otherwise.  Returns SKIM_OK, or 1 when the
// call does not meet the kernel's requirements (then the generic sort kernel must be used).
int skim_launch_sort16(skim_ctx *ctx, skimk::ClusterArgs &args, int64_t rows, bool launch);
// Lloyd kernel (skim_lloyd.cu): one warp per row record.
int skim_launch_lloyd(skim_ctx *ctx, const skimk::ClusterArgs &args, int64_t rows);
