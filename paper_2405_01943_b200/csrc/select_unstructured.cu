// Unstructured DaSS selection at a sparsity ratio s (Section 3, "Pruning Granularity"): in every comparison
// line -- a column of Wg / Wu (all neurons at one input: input-balanced) or a row of Wd (output-balanced) --
// the floor(s * L) weights with the lowest Eq. 4 / Eq. 5 score are pruned.  No sort.
//
// The order of the oracle, "higher score first, lower index first", is the order of a three-part key: the
// rounded product fl32(|w| * scale), then the exact double product, then the index counted from the top.
//
// Lines of FAST_MIN_L elements and more are decided by two streaming sweeps: 1024 evenly spaced elements of the line
// give, through two small histograms (no sort), a bracket of rounded products that holds the cut unless the sample is
// five standard deviations off; the first sweep reduces every element into a 1024-bin histogram of the bracket (those
// outside land on idle words) and counts the elements below it; one warp finds the bin that holds the cut; the second
// sweep writes the outputs -- above the bin stays, below it goes -- and sets the bin's few elements aside; one warp
// ranks those by the full key and puts the survivors back.  A line whose bracket misses, or whose bin holds more than
// CAND_CAP elements, is decided by the radix select: the k-th largest key is found 11 bits at a time with
// shared-memory histograms, and a line stops as soon as the bucket at the cut holds exactly the survivors still
// wanted (exact products and indices are consulted only where rounded products tie across the cut).
//
// Lines that are matrix rows: select_rows_stream_kernel (both sweeps, two rows per CTA), then select_rows_kernel
// (radix select, the row cached in shared memory) for the rows the first kernel listed, or for every row when the
// lines are short.  Lines that are matrix columns: select_cols_kernel (one CTA per strip of 8 adjacent columns: sample,
// first sweep, bin; radix select inside the kernel where needed) publishes a LineResult per column, a streaming
// kernel with coalesced rows emits (select_emit_stream_kernel for bf16, select_emit_cols_kernel for f32), and
// select_fix_cols_kernel ranks what the emit pass set aside.
#include "select_common.cuh"

namespace dass {

// out[i] = fl32(norm[i]^alpha) for i < n, 0 for the padding up to npad (a multiple of 8, so that the selection
// kernel can read whole 8-element chunks)
__global__ void scale_vector_kernel(const float *__restrict__ norm, int64_t n, int64_t npad, int mode, float alpha,
                                    float *__restrict__ out)
{
    const int64_t i = (int64_t)blockIdx.x * blockDim.x + threadIdx.x;
    if (i < n) DASS_ST(&out[i], scale_from_norm(DASS_LD(&norm[i]), mode, alpha));
    else if (i < npad) DASS_ST(&out[i], 0.0f);
}


size_t select_results_bytes(int64_t cols) { return ((size_t)cols * sizeof(LineResult) + 31) / 32 * 32; }
size_t select_scale_bytes(int64_t n) { return (size_t)((n + 7) / 8 * 8) * sizeof(float); }
// [per-column results][scale vector padded to 8][count of undecided rows, 32 bytes][their indices]
// [per column: count of elements set aside][their keys][rows][stored weights]
size_t select_workspace_bytes(int64_t rows, int64_t cols, bool norm_cols)
{
    return select_results_bytes(cols) + select_scale_bytes(norm_cols ? cols : rows) + 32 + (size_t)((rows + 7) / 8 * 8) * sizeof(uint32_t) +
           (size_t)((cols + 7) / 8 * 8) * sizeof(uint32_t) * (1 + 3 * CAND_CAP);
}

cudaError_t select_unstructured_launch(const void *W, int64_t rows, int64_t cols, int64_t ld, bool bf16,
                                       const float *norm, bool norm_cols, float alpha, uint32_t k, bool line_is_row,
                                       uint32_t *mask_bits, void *W_pruned, void *workspace, cudaStream_t st)
{
    LineResult *results = static_cast<LineResult *>(workspace);
    float *scale_ws = reinterpret_cast<float *>(static_cast<unsigned char *>(workspace) + select_results_bytes(cols));
    const int64_t n_norm = norm_cols ? cols : rows;
    uint32_t *line_count = reinterpret_cast<uint32_t *>(reinterpret_cast<unsigned char *>(scale_ws) + select_scale_bytes(n_norm));
    uint32_t *line_list = line_count + 8;
    const size_t cols8 = (size_t)((cols + 7) / 8 * 8);
    CandLists cand;
    cand.count = line_list + (rows + 7) / 8 * 8;
    cand.key = cand.count + cols8;
    cand.idx = cand.key + cols8 * CAND_CAP;
    cand.raw = cand.idx + cols8 * CAND_CAP;
    const int64_t n_pad = (n_norm + 7) / 8 * 8;
    scale_vector_kernel<<<(unsigned)((n_pad + 255) / 256), 256, 0, st>>>(norm, n_norm, n_pad, (int)scale_mode_for(alpha), alpha, scale_ws);
    cudaError_t e = cudaGetLastError();
    if (e != cudaSuccess) return e;
    SelectParams p;
    p.W = W; p.Wp = W_pruned; p.mask = mask_bits; p.scale = scale_ws; p.results = results;
    p.line_count = nullptr; p.line_list = nullptr;
    p.cand_count = (!line_is_row && bf16) ? cand.count : nullptr;
    p.status = stage_b_status_word();
    p.rows = rows; p.cols = cols; p.ld = ld;
    p.wpr = (cols + 31) / 32;
    p.L = line_is_row ? cols : rows;
    p.lpad = (p.L + 7) / 8 * 8;
    p.k = k;
    p.idx_bits = 1;
    while (((int64_t)1 << p.idx_bits) < p.L) ++p.idx_bits;
    p.scale_along_line = (line_is_row == norm_cols) ? 1 : 0;   // the norm index runs along the line
    {   // five standard deviations of the rank of a sample quantile, in sample positions, plus slack: a line in
        // two million misses (a column that misses sends its whole strip of eight through the radix select, which
        // can lengthen the launch by a CTA's radix passes; the wider bracket costs nothing, every element is reduced
        // into a counter either way)
        const double q = (double)(p.L - (int64_t)k) / (double)p.L;
        p.margin = (int)std::ceil(5.0 * std::sqrt((double)SELECT_SAMPLE * q * (1.0 - q))) + 2;
    }
    if (line_is_row) {
        if (mask_bits) {   // the kernel writes whole bytes of real columns; the padding of each mask row must read 0
            e = cudaMemsetAsync(mask_bits, 0, (size_t)rows * p.wpr * sizeof(uint32_t), st);
            if (e != cudaSuccess) return e;
        }
        return select_launch_rows(p, bf16, line_count, line_list, st);
    }
    e = select_launch_cols(p, bf16, st);
    if (e != cudaSuccess) return e;
    return select_launch_emit(p, bf16, cand, norm_cols ? 0 : 1, st);
}

}  // namespace dass

using namespace dass;

extern "C" dass_status dass_select_workspace_bytes(int64_t rows, int64_t cols, dass_axis norm_axis, size_t *bytes)
{
    if (!bytes) return DASS_ERR_NULL;
    if (norm_axis != DASS_AXIS_ROWS && norm_axis != DASS_AXIS_COLS) return DASS_ERR_DTYPE;
    if (rows < 1 || cols < 1) return DASS_ERR_SHAPE;
    *bytes = select_workspace_bytes(rows, cols, norm_axis == DASS_AXIS_COLS);
    return DASS_OK;
}

extern "C" dass_status dass_select_unstructured(const void *W, int64_t rows, int64_t cols, int64_t ld, dass_dtype dt,
                                                const float *norm, dass_axis norm_axis, float alpha,
                                                double sparsity, dass_axis compare_axis,
                                                uint32_t *mask_bits, void *W_pruned,
                                                void *workspace, size_t workspace_bytes, void *cuda_stream)
{
    if (!W || !norm || (!mask_bits && !W_pruned)) return DASS_ERR_NULL;
    if (dt != DASS_BF16 && dt != DASS_F32) return DASS_ERR_DTYPE;
    if ((norm_axis != DASS_AXIS_ROWS && norm_axis != DASS_AXIS_COLS) ||
        (compare_axis != DASS_AXIS_ROWS && compare_axis != DASS_AXIS_COLS)) return DASS_ERR_DTYPE;
    if (rows < 1 || cols < 1 || ld < cols) return DASS_ERR_SHAPE;
    if (!(sparsity >= 0.0 && sparsity < 1.0)) return DASS_ERR_SHAPE;
    if (!std::isfinite(alpha) || alpha < 0.0f) return DASS_ERR_UNSUPPORTED;
    const bool bf16 = dt == DASS_BF16;
    if (ld % (bf16 ? 8 : 4) != 0) return DASS_ERR_ALIGN;
    if ((reinterpret_cast<uintptr_t>(W) & 15u) || (W_pruned && (reinterpret_cast<uintptr_t>(W_pruned) & 15u)) ||
        (reinterpret_cast<uintptr_t>(norm) & 3u) || (reinterpret_cast<uintptr_t>(mask_bits) & 3u)) return DASS_ERR_ALIGN;
    const bool line_is_row = compare_axis == DASS_AXIS_COLS;         // the index that varies inside a line
    const int64_t L = line_is_row ? cols : rows;
    if (L >= (int64_t)1 << 31) return DASS_ERR_UNSUPPORTED;
    if (line_is_row && select_row_smem_bytes(L, bf16) > (size_t)220 * 1024) return DASS_ERR_UNSUPPORTED;   // a row line is cached in shared memory
    size_t need = 0;
    const dass_status qs = dass_select_workspace_bytes(rows, cols, norm_axis, &need);
    if (qs != DASS_OK) return qs;
    if (!workspace || workspace_bytes < need) return DASS_ERR_WORKSPACE;
    if (reinterpret_cast<uintptr_t>(workspace) & 15u) return DASS_ERR_ALIGN;
    const int64_t n_prune = (int64_t)std::floor(sparsity * (double)L);
    const uint32_t k = (uint32_t)(L - n_prune);
    DASS_BOUNDS_SCOPE(bs);
    DASS_BOUNDS_ADD(bs, W, (size_t)rows * ld * (bf16 ? 2 : 4));
    DASS_BOUNDS_ADD(bs, W_pruned, (size_t)rows * ld * (bf16 ? 2 : 4));
    DASS_BOUNDS_ADD(bs, norm, (size_t)(norm_axis == DASS_AXIS_ROWS ? rows : cols) * sizeof(float));
    DASS_BOUNDS_ADD(bs, mask_bits, (size_t)rows * ((cols + 31) / 32) * sizeof(uint32_t));
    DASS_BOUNDS_ADD(bs, workspace, workspace_bytes);
    DASS_BOUNDS_COMMIT(bs, static_cast<cudaStream_t>(cuda_stream));
    if (select_unstructured_launch(W, rows, cols, ld, bf16, norm, norm_axis == DASS_AXIS_COLS, alpha, k, line_is_row,
                                   mask_bits, W_pruned, workspace,
                                   static_cast<cudaStream_t>(cuda_stream)) != cudaSuccess)
        return DASS_ERR_CUDA;
    return DASS_OK;
}
