// Tensor-core (tcgen05) dense products for bf16 operands.
#pragma once

#include "common.cuh"

namespace e2egrec {

// h' = act(cat W^T + b) for `rows` (a multiple of 128) rows of cat [rows x k] and W [n x k], both bf16
// row-major; rows at and beyond *m_dev inside a partly used 128-row tile are written as zeros, tiles
// wholly beyond it are left alone.  `status` receives E2EGREC_DEV_TIMEOUT if a bounded wait runs out.
// Returns false when the shape is outside what the kernel takes, in which case nothing was enqueued.
// out2 (optional, [rows2 x ldo2]): the rows below rows2 of every written tile are stored there as well.
bool tc_update_forward(const __nv_bfloat16 *cat, int64_t rows, int k, const __nv_bfloat16 *W, int n, const float *bias,
                       int relu, __nv_bfloat16 *out, const int32_t *m_dev, int32_t *status, cudaStream_t st,
                       __nv_bfloat16 *out2 = nullptr, int64_t ldo2 = 0, int64_t rows2 = 0);

// Eq. 2 and Eq. 3 of one layer in one launch (bf16, d_in of 64, 128 or 256 values, n <= 256 a multiple of 32):
//   cat[i] = [ Hsrc[self_ids ? self_ids[i] : i] | mean over k in [indptr[i], indptr[i+1]) of Hsrc[nbr[k]] ]   (stored for the
//   backward pass, zero rows from *m_dev up to the next multiple of 128),   out = act(cat W^T + bias)
// with the rows of cat built in shared memory as the A operand, never read back from global memory.  Same conventions and
// the same bits as sage_aggregate_kernel followed by tc_update_forward.
bool tc_sage_fused_forward(const __nv_bfloat16 *Hsrc, int64_t ld, const int32_t *nbr, const int32_t *self_ids,
                           const int32_t *indptr, int d_in, __nv_bfloat16 *cat, int64_t rows, const __nv_bfloat16 *W, int n,
                           const float *bias, int relu, __nv_bfloat16 *out, const int32_t *m_dev, int32_t *status,
                           cudaStream_t st, __nv_bfloat16 *out2 = nullptr, int64_t ldo2 = 0, int64_t rows2 = 0);

// dCat = dZ W with the layer weight W [d_out x 2 d_in] as stored (the tensor cores read it with its N index
// contiguous, no transposed copy is made); columns >= d_in are scaled by inv_cnt[row].  2 d_in must be a multiple
// of 64.  Same conventions as above.
// n_rhs > 1: dz and dcat hold n_rhs blocks of `rows` rows each (several gradients sent through the layer in one pass), the
// first *m_dev rows of every block live; inv_cnt is indexed by the row inside its block.
bool tc_dcat_backward(const __nv_bfloat16 *dz, int64_t rows, int d_out, const __nv_bfloat16 *W, int two_d_in,
                      const float *inv_cnt, __nv_bfloat16 *dcat, const int32_t *m_dev, int32_t *status, cudaStream_t st,
                      int n_rhs = 1);

// Optional forms of the product's epilogue (all matrices [rows x n], bf16, 16-byte aligned rows):
//   gate_in  F:  out = g * F with g = sigmoid(product + bias); the pre-activation and g are rounded to bf16 first,
//                and g is stored to gate_out as well when that is given (gating fusion, Sec. 4.3.2);
//   add_a, add_b: out = round_bf16(product) + add_a * add_b, element by element (the gate's input gradient).
struct TcFuse {
    const __nv_bfloat16 *gate_in;
    int64_t ld_gate_in;
    __nv_bfloat16 *gate_out;
    int64_t ld_gate_out;
    const __nv_bfloat16 *add_a, *add_b;
    int64_t ld_add_a, ld_add_b;
};

// out = mask * act(A B^T + bias): A [rows x k], B [n x k], out [rows x ldo], optional mask [rows x ld_mask]
// (outputs zeroed where mask <= 0).  With b_is_k_by_n, B is given as [k x n] row-major instead (out = A B; n a
// multiple of 64).  Same conventions as above.
bool tc_linear(const __nv_bfloat16 *A, int64_t rows, int k, const __nv_bfloat16 *B, int n, const float *bias, int relu,
               const __nv_bfloat16 *mask, int64_t ld_mask, __nv_bfloat16 *out, int64_t ldo, const int32_t *m_dev,
               int32_t *status, cudaStream_t st, bool b_is_k_by_n = false, const TcFuse *fuse = nullptr);

// part[z] = (rows of split z of dY)^T (same rows of Xin): dY [rows x m], Xin [rows x n] bf16 row-major, part
// [splits x m x n] fp32.  Rows between *m_dev and the next multiple of 64 must be zero in both matrices.
// n_rhs > 1: dY holds n_rhs blocks of `rows` rows that all meet the same `rows` rows of Xin; the result is the sum over them.
bool tc_weight_grad(const __nv_bfloat16 *dY, int64_t rows, int m, const __nv_bfloat16 *Xin, int n, const int32_t *m_dev,
                    float *part, int splits, int32_t *status, cudaStream_t st, int n_rhs = 1);
// Output tiles (128 x up to 256) of tc_weight_grad for an m x n result: gridDim.x * gridDim.y of its launch.
int tc_weight_grad_tiles(int m, int n);

}  // namespace e2egrec
