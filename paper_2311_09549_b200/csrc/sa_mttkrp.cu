// Kernel 8 <MTTKRP,GEMM>:  A(i,m) = sum_{j,k,r} B(i,j,k) C(j,r) D(k,r) E(r,m)  (Table of kernels, Section 6,
// Description column in this library's letters: B order-3 CSF, C and D the factor matrices of the MTTKRP,
// E the weight matrix of the GEMM).  Branched nest
//   i < T(r) ;  j' < t(r) ; k': t(r) += B(i,j,k) D(k,r) ,  r: T(r) += t(r) C(j,r) > ,  m,r: A(i,m) += T(r) E(r,m) >
// The inner pair is the fiber stage of kernel 6 with an element-wise consumer instead of the outer product
// (sa_ttm3.cu, template flag HAD); the rows T(i,:) pass through the workspace and the dense stage is the
// BF16x3 tensor-core GEMM shared with kernels 2 and 4.
#include "sa_device.cuh"

sa_status sa_launch_mttkrp_rows(const sa_tensor *t, const sa_dense &C, const sa_dense &D, float *out, float *partial,
                                cudaStream_t stream, int *launches);

bool sa_ranks_ok_mttkrp_gemm(int64_t R, int64_t M) { return R == 32 && sa_dense_gemm_ok(R, M); }

// workspace: [T: I x R][partial rows of split slices]
size_t sa_ws_mttkrp_gemm(const sa_tensor *t, const sa_dense *ops)
{
    const size_t R = size_t(ops[0].cols);
    return sa_align256(size_t(t->dims[0]) * R * sizeof(float)) + sa_align256(size_t(t->wl_main.n_slots) * R * sizeof(float));
}

sa_status sa_launch_mttkrp_gemm(const sa_tensor *t, const sa_dense *ops, float *out, void *ws, size_t, cudaStream_t stream,
                                int *launches)
{
    const int64_t I = t->dims[0], R = ops[0].cols, M = ops[2].cols;
    float *T = static_cast<float *>(ws);
    float *partial = reinterpret_cast<float *>(static_cast<char *>(ws) + sa_align256(size_t(I) * size_t(R) * sizeof(float)));
    int n1 = 0;
    sa_status s = sa_launch_mttkrp_rows(t, ops[0], ops[1], T, partial, stream, &n1);
    if (s != SA_OK) return s;
    s = sa_launch_dense_gemm(I, T, R, ops[2].ptr, ops[2].ld, R, M, out, t->d_status, stream);
    if (s != SA_OK) return s;
    *launches = n1 + 1;
    return SA_OK;
}
