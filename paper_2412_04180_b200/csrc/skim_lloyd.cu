// Lloyd kernel, the second half of the row clustering (SKIM Algorithm 3, error pre-recording loop;
// objective of Section 3.2, diagonal form): one warp per row iterates on the row record the sort
// kernel left in global memory (sorted keys and importance, group index, binary64 block prefix sums)
// and writes the row's centroids and error table entries.
//
// An iteration is a chain of dependent small steps (midpoint, search, a few loads, a quotient), so a
// single row cannot go fast; the kernel gets its throughput from the number of rows in flight: 32 warps
// per SM, each on its own row.  Per iteration a lane touches a 32-byte window of the group index and one
// 64-byte group record (8 keys, 8 importances, two prefix sums); these move slowly from one iteration to
// the next and are served by L1 through the read-only path.
#include "skim_cluster_phases.cuh"

namespace {

using namespace skimk;

constexpr int LLOYD_WARPS = 4;   // rows per block

template <typename KeyT>
__global__ void __launch_bounds__(LLOYD_WARPS * 32, 8) skim_lloyd_kernel(ClusterArgs a, int rows_in_chunk)
{
    __shared__ PhaseSmem ps_all[LLOYD_WARPS];
    const int warp = threadIdx.x >> 5, lane = threadIdx.x & 31;
    const int local = blockIdx.x * LLOYD_WARPS + warp;
    if (local >= rows_in_chunk) return;
    PhaseSmem &ps = ps_all[warp];
    const int64_t row = a.row0 + local;
    const unsigned char *rec = a.scratch + (size_t)local * (size_t)a.rec_stride;
    const int nd = *reinterpret_cast<const int *>(rec);
    if (lane < 16) ps.dvals[lane] = reinterpret_cast<const float *>(rec + 64)[lane];
    __syncwarp();
    lloyd_warp<KeyT>(rec, nd, a, row, ps);
    if (!a.codes) return;
    __syncwarp();
    write_codes(a, row, ps, lane, 32);
}

}  // namespace

int skim_launch_lloyd(skim_ctx *ctx, const ClusterArgs &args, int64_t rows, int key_bytes)
{
    const unsigned blocks = (unsigned)((rows + LLOYD_WARPS - 1) / LLOYD_WARPS);
    if (key_bytes == 2)
        skim_lloyd_kernel<uint16_t><<<blocks, LLOYD_WARPS * 32, 0, ctx->stream>>>(args, (int)rows);
    else
        skim_lloyd_kernel<uint32_t><<<blocks, LLOYD_WARPS * 32, 0, ctx->stream>>>(args, (int)rows);
    SKIM_CUDA_OK(cudaGetLastError());
    ctx->launches += 1;
    return SKIM_OK;
}
