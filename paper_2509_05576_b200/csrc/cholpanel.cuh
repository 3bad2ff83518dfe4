// Upper Cholesky of a large matrix in panels: the cooperative float64 kernel factorises a panel of kPanelBlocks block
// rows (touching only those rows), then the panel is applied to everything below it in one product of depth
// 64 kPanelBlocks on the int8 tensor path (i8gemm.cuh),
//     A[i][j] -= sum_{r in panel} U[r][i] U[r][j]   (i, j below the panel, upper tiles),
//     W[i][c] -= sum_{r in panel} U[r][i] W[r][c]   (i below the panel, c up to its end),
// instead of one 64-deep float64 MMA update per block row: with a depth of 1024 the product moves a small fraction of the bytes
// per multiply-add through L2.  The blocked form of Eq. 12 / Sec. 5 item 1 is unchanged, only the grouping of the updates.
#pragma once
#include "chol.cuh"
#include "i8gemm.cuh"

namespace ptq {

constexpr int kPanelBlocks = 16;             // 1024 columns per panel
constexpr int kPanelMinCols = 3072;          // below this the single cooperative launch is faster

inline size_t chol_panel_workspace_bytes(int n) {
    if (n < kPanelMinCols) return 0;
    return 2 * x_operand_bytes(n, kPanelBlocks * kNB);
}

// Same contract as cholesky_upper (whole factorisation); xws: chol_panel_workspace_bytes(n) bytes of scratch.
inline int cholesky_upper_auto(double* A, int n, double* Wm, double* Dbuf, unsigned* bar, void* xws, int32_t* status,
                               cudaStream_t stream) {
    if (n < kPanelMinCols || xws == nullptr) return cholesky_upper(A, n, Wm, Dbuf, bar, status, stream);
    const int nb = (n + kNB - 1) / kNB;
    for (int kf = 0; kf < nb; kf += kPanelBlocks) {
        const int pe = kf + kPanelBlocks < nb ? kf + kPanelBlocks : nb;
        int st = cholesky_upper(A, n, Wm, Dbuf, bar, status, stream, pe, kf, pe);
        if (st) return st;
        if (pe >= nb) break;
        const int r0 = kf * kNB, c0 = pe * kNB;               // panel rows r0 .. c0 - 1, everything from c0 on is below it
        const int depth = c0 - r0, rest = n - c0;
        Carver cv(xws);
        // rows of the operand = columns c0 .. n - 1 of the panel's rows of U
        const XOperand u = x_slice_operand(cv, A + (size_t)r0 * n + c0, n, 1, rest, depth, stream);
        XGemmParams prm{};
        prm.C = A + (size_t)c0 * n + c0; prm.ldc = n; prm.alpha = -1.0; prm.status = status;
        prm.out_mode = X_OUT_ADD_UPPER; prm.k_mode = X_K_ALL;
        st = x_product(u, u, prm, stream);
        if (st) return st;
        if (Wm != nullptr) {
            // rows of the operand = columns 0 .. c0 - 1 of the panel's rows of W
            const XOperand w = x_slice_operand(cv, Wm + (size_t)r0 * n, n, 1, c0, depth, stream);
            prm.C = Wm + (size_t)c0 * n; prm.out_mode = X_OUT_ADD;
            st = x_product(u, w, prm, stream);
            if (st) return st;
        }
    }
    return PTQ_OK;
}

}  // namespace ptq
