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
// multiples of 16 bytes.
//   hdr     int nd (number of distinct values) at byte 0; double totals[3] (sum g, sum g x,
//           sum g x^2 over the row) at byte 16; float dvals[16] at byte 64
//   groups  one record per group of 8 sorted elements: 8 keys, 8 importances, and the binary64
//           exclusive prefix sums of g and g*x at the group's first element.  Everything a boundary
//           needs in one Lloyd iteration sits in these 64 (16-bit keys) or 80 (32-bit keys) bytes.
//           The last group is padded with the largest key and zero importance.
//   gi      group index: first key of every group, sk_entries(m) keys (padded with the largest key)
//   p2      binary64 exclusive prefix sums of g*x^2 at every group start (ngrp + 1 entries), read
//           once, for the error
struct RowRecord {
    size_t groups, gi, p2, total;
    size_t group_bytes, gi_bytes, p2_bytes;
    int ngrp;
};

__host__ __device__ inline int sk_entries(int m) { return ((((m + 7) >> 3) + 7) & ~7) + 16; }

__host__ __device__ inline RowRecord row_record(int m, int key_bytes)
{
    RowRecord R;
    R.ngrp = (m + 7) >> 3;
    R.group_bytes = (size_t)8 * key_bytes + 32 + 16;
    R.gi_bytes = (size_t)sk_entries(m) * key_bytes;
    R.p2_bytes = ((size_t)(R.ngrp + 1) * 8 + 15) & ~(size_t)15;
    size_t off = 128;
    R.groups = off; off += (size_t)R.ngrp * R.group_bytes;
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
    double errs[32];
    float tfs[32];
    float dvals[32];
    int misc[4];   // [0] distinct count, [1] slot counter
};

// An aligned group of 8 sorted elements (keys and importance) held in registers.
template <typename KeyT> struct Group8;

template <> struct Group8<uint16_t> {
    uint4 kv;
    float4 ga, gb;
    // from a group record in global memory (read-only path); also returns its two prefix sums
    __device__ __forceinline__ double2 load_record(const unsigned char *gr)
    {
        kv = __ldg(reinterpret_cast<const uint4 *>(gr));
        ga = __ldg(reinterpret_cast<const float4 *>(gr + 16));
        gb = __ldg(reinterpret_cast<const float4 *>(gr + 32));
        return __ldg(reinterpret_cast<const double2 *>(gr + 48));
    }
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
    __device__ __forceinline__ double2 load_record(const unsigned char *gr)
    {
        ka = __ldg(reinterpret_cast<const uint4 *>(gr));
        kb = __ldg(reinterpret_cast<const uint4 *>(gr + 16));
        ga = __ldg(reinterpret_cast<const float4 *>(gr + 32));
        gb = __ldg(reinterpret_cast<const float4 *>(gr + 48));
        return __ldg(reinterpret_cast<const double2 *>(gr + 64));
    }
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

// Group index: GI[q] = first key of the q-th group of 8 sorted elements, padded with the largest
// key to sk_entries(m) entries.  The boundary search of the Lloyd iteration runs over this 8x
// smaller array first.
template <typename KeyT, int THREADS>
__device__ __forceinline__ void build_group_index(const KeyT *skeys, int m, KeyT *GI)
{
    const int ngrp = (m + 7) >> 3, n = sk_entries(m);
    for (int q = threadIdx.x; q < n; q += THREADS) GI[q] = q < ngrp ? skeys[q << 3] : KeyOps<KeyT>::PAD;
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
// to whole groups, group index, block prefix sums).  Call with all threads, after
// block_prefix_sums (and collect_distinct when nd <= 16).
template <typename KeyT, int THREADS>
__device__ __forceinline__ void write_row_record(const ClusterArgs &a, const KeyT *skeys, const float *sg, const KeyT *GI,
                                                 const double *PB, int nd, const float *dvals)
{
    const RowRecord R = row_record(a.m, (int)sizeof(KeyT));
    unsigned char *rec = a.scratch + (size_t)blockIdx.x * (size_t)a.rec_stride;
    const int BLK = 1 << a.blk_shift;
    const int nblk = (a.m + BLK - 1) >> a.blk_shift;
    const double *PB0 = PB, *PB1 = PB + (nblk + 1), *PB2 = PB + 2 * (nblk + 1);
    if (threadIdx.x == 0) {
        *reinterpret_cast<int *>(rec) = nd;
        double *tot = reinterpret_cast<double *>(rec + 16);
        tot[0] = PB0[nblk]; tot[1] = PB1[nblk]; tot[2] = PB2[nblk];
    }
    if (threadIdx.x < 16) reinterpret_cast<float *>(rec + 64)[threadIdx.x] = nd <= 16 ? dvals[threadIdx.x] : 0.0f;
    double *p2 = reinterpret_cast<double *>(rec + R.p2);
    for (int q = threadIdx.x; q <= R.ngrp; q += THREADS) {
        // prefix sums at the start of group q: the block's entry plus the whole groups before q in it
        if (q == R.ngrp) { p2[q] = PB2[nblk]; break; }
        const int e = q << 3;
        const int blk = e >> a.blk_shift;
        D3 P = {PB0[blk], PB1[blk], PB2[blk]};
        for (int u = blk << a.blk_shift; u < e; u += 8) add_group8<KeyT, true>(skeys + u, sg + u, 8, P);
        p2[q] = P.c;
        {
            unsigned char *gr = rec + R.groups + (size_t)q * R.group_bytes;
            constexpr int KB = 8 * (int)sizeof(KeyT);
            const uint4 *ks = reinterpret_cast<const uint4 *>(skeys + (q << 3));
            uint4 *kd = reinterpret_cast<uint4 *>(gr);
#pragma unroll
            for (int u = 0; u < KB / 16; ++u) kd[u] = ks[u];
            const uint4 *gsrc = reinterpret_cast<const uint4 *>(sg + (q << 3));
            uint4 *gd = reinterpret_cast<uint4 *>(gr + KB);
            gd[0] = gsrc[0];
            gd[1] = gsrc[1];
            *reinterpret_cast<double2 *>(gr + KB + 32) = make_double2(P.a, P.b);
        }
    }
    copy16<THREADS>(rec + R.gi, GI, R.gi_bytes);
}

// A window of 16 ascending keys of the group index around the previous boundary position (at
// least 4 entries, i.e. 32 elements, on either side), held in registers across one Lloyd
// iteration: the next search needs no shared-memory round trip unless the boundary left it.
template <typename KeyT> struct KeyWindow;

template <> struct KeyWindow<uint16_t> {
    static constexpr int N = 16;
    uint4 v[2];
    int ws;
    __device__ __forceinline__ void load(const uint16_t *skeys, int m, int guess)
    {
        const int top = ((m + 7) & ~7) - N;
        ws = max(0, min((((guess + 4) >> 3) << 3) - 8, top));
        const uint4 *p = reinterpret_cast<const uint4 *>(skeys + ws);
        v[0] = __ldg(p); v[1] = __ldg(p + 1);
    }
    // number of window keys <= kt.  A word holds two ascending keys (low half first), so
    // "high half <= kt" is one 32-bit compare against (kt << 16 | 0xffff) and "low half <= kt"
    // one compare of the word shifted left by 16.
    __device__ __forceinline__ int count_le(uint16_t kt) const
    {
        const uint32_t khi = ((uint32_t)kt << 16) | 0xffffu, klo = (uint32_t)kt << 16;
        const uint32_t w[8] = {v[0].x, v[0].y, v[0].z, v[0].w, v[1].x, v[1].y, v[1].z, v[1].w};
        int c = 0;
#pragma unroll
        for (int q = 0; q < 8; ++q) c += (w[q] <= khi ? 1 : 0) + ((w[q] << 16) <= klo ? 1 : 0);
        return c;
    }
};

template <> struct KeyWindow<uint32_t> {
    static constexpr int N = 16;
    uint4 v[4];
    int ws;
    __device__ __forceinline__ void load(const uint32_t *skeys, int m, int guess)
    {
        const int top = ((m + 7) & ~7) - N;
        ws = max(0, min((((guess + 4) >> 3) << 3) - 8, top));
        const uint4 *p = reinterpret_cast<const uint4 *>(skeys + ws);
#pragma unroll
        for (int q = 0; q < 4; ++q) v[q] = __ldg(p + q);
    }
    __device__ __forceinline__ int count_le(uint32_t kt) const
    {
        int c = 0;
#pragma unroll
        for (int q = 0; q < 4; ++q)
            c += (v[q].x <= kt ? 1 : 0) + (v[q].y <= kt ? 1 : 0) + (v[q].z <= kt ? 1 : 0) + (v[q].w <= kt ? 1 : 0);
        return c;
    }
};

// s1 / s0 for s0 > 0: binary32 reciprocal seed and two binary64 Newton corrections (relative
// error about 2^-60, i.e. the correctly rounded quotient up to the last bit or so); operands far
// outside the binary32 range take the plain division.
__device__ __forceinline__ double quotient(double s1, double s0)
{
    const float s0f = (float)s0;
    if (!(s0f > 1e-30f && s0f < 1e30f) || !(fabs(s1) < 1e30)) return s1 / s0;
    const float rf = __frcp_rn(s0f);
    const double rd = (double)rf;
    double q = (double)((float)s1 * rf);
    q = fma(fma(-q, s0, s1), rd, q);
    q = fma(fma(-q, s0, s1), rd, q);
    return q;
}

// Lloyd iterations and the error table entry of one row, run by ONE warp on the row record in
// global memory (all 32 lanes must call).
// Lane L owns centroid L of the row's concatenated centroid record and the boundary above it.
// Per iteration a lane: forms the exact midpoint; counts the group-index entries below it in a
// register window prefetched around the previous position (falling back to a binary search of the
// group index when the boundary left the window); loads that one group record, which gives the
// exact boundary position (keys), the prefix sums at the group start and the few elements between.
// On return ps.tfs[L] holds the boundary (largest binary32 value still assigned to centroid L).
template <typename KeyT>
__device__ __forceinline__ void lloyd_warp(const unsigned char *rec, int nd, const ClusterArgs &a, int64_t row, PhaseSmem &ps)
{
    using K = KeyOps<KeyT>;
    using Win = KeyWindow<KeyT>;
    const int lane = threadIdx.x & 31;
    const int m = a.m;
    const RowRecord R = row_record(m, (int)sizeof(KeyT));
    const unsigned char *groups = rec + R.groups;
    const KeyT *GI = reinterpret_cast<const KeyT *>(rec + R.gi);
    const double *P2 = reinterpret_cast<const double *>(rec + R.p2);
    const double *tot = reinterpret_cast<const double *>(rec + 16);
    const int ngi = sk_entries(m) - 16;                 // group-index entries up to the padding margin
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
    const bool searches = normal && j < k - 1;
    float c = 0.0f;
    if (degenerate) c = ps.dvals[min(j, nd - 1)];
    if (normal) {
        const int idx = (int)(((long long)(2 * j + 1) * m) / (2 * k));
        c = K::to_float(reinterpret_cast<const KeyT *>(groups + (size_t)(idx >> 3) * R.group_bytes)[idx & 7]);
    }
    const double tot0 = normal ? tot[0] : 0.0, tot1 = normal ? tot[1] : 0.0;

    int Bprev = -1;
    float tf = __int_as_float(0x7f800000);            // +inf: no boundary above the last centroid
    double err_j = 0.0;
    Win win;
    win.ws = 0;
    bool have_win = false;
    for (int it = 0;; ++it) {
        const float c_up = __shfl_down_sync(0xffffffffu, c, 1);
        int B = m, grp_i = 0, cntk = 0;
        Group8<KeyT> grp;
        double2 gp = make_double2(0.0, 0.0);          // prefix sums at the group start
        if (has_boundary) {
            // exact midpoint of two binary32 centroids, rounded down to binary32: x <= midpoint
            // holds for a binary32 x exactly when x <= tf
            tf = __double2float_rd(0.5 * ((double)c + (double)c_up));
            if (tf == 0.0f) tf = 0.0f;
        }
        if (searches) {
            const KeyT kt = K::floor_key(tf);
            int nle = -1;                              // group-index entries <= kt
            if (have_win) {
                const int cnt = win.count_le(kt);
                if ((cnt > 0 || win.ws == 0) && cnt < Win::N) nle = win.ws + cnt;
            }
            if (nle < 0) {
                int lo = 0, hi = ngi;
                while (lo < hi) {
                    const int mid = (lo + hi) >> 1;
                    if (__ldg(GI + mid) <= kt) lo = mid + 1; else hi = mid;
                }
                nle = lo;
            }
            grp_i = max(nle - 1, 0);
            gp = grp.load_record(groups + (size_t)grp_i * R.group_bytes);
            cntk = grp.count_le(kt);
            B = min((grp_i << 3) + cntk, m);
        }
        const bool same = __all_sync(0xffffffffu, B == Bprev);
        const bool final = (it >= a.iters) || same;
        Bprev = B;
        D3 P = {0.0, 0.0, 0.0};
        if (normal) {
            if (searches) {
                P.a = gp.x;
                P.b = gp.y;
                if (final) {
                    P.c = __ldg(P2 + grp_i);
                    add_group<KeyT, true>(grp, cntk, P);
                } else {
                    add_group<KeyT, false>(grp, cntk, P);
                    win.load(GI, ngi, grp_i + 1);       // for the next iteration
                    have_win = true;
                }
            } else {
                // the last centroid of a width has no boundary above it: its prefix is the row total
                P.a = tot0;
                P.b = tot1;
                if (final) P.c = tot[2];
            }
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
        if (normal && S0 > 0.0) c = (float)quotient(S1, S0);
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
__device__ __forceinline__ void write_codes(const ClusterArgs &a, int64_t row, const PhaseSmem &ps, int start, int stride)
{
    const int m = a.m;
    const uint16_t *Wr = a.W + row * a.ld;
    int only = -1;
    if (a.row_bits) only = (int)a.row_bits[row] - a.bmin;
    for (int e = start; e < m; e += stride) {
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

// fp16-key sort kernel (skim_cluster16.cu).  Fills *blk_shift and *rec_bytes when `launch` is false
// (planning) and launches over `rows` rows otherwise.  Returns SKIM_OK, or 1 when the call does not
// meet the kernel's requirements (then the generic sort kernel must be used).
int skim_launch_sort16(skim_ctx *ctx, skimk::ClusterArgs &args, int64_t rows, bool launch);
// Lloyd kernel (skim_lloyd.cu): one warp per row record.
int skim_launch_lloyd(skim_ctx *ctx, const skimk::ClusterArgs &args, int64_t rows, int key_bytes);
