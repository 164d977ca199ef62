"""Algorithm 1 of the paper (Grouped Spatial Pack Convolutions) restated in numpy, as a second,
structurally different CPU implementation used only to cross-check the oracle.

The four stages are taken in the paper's order: kernel reshaping into the 7-D volume
[g, KPG/T_O, CPG/T_I, K_h, K_w, T_I, T_O], input reshaping of the zero-padded input into the 6-D
volume [g, N, CPG/T_I, H_i, T_I, W_i], the convolution on the 6-D output volume
[g, N, KPG/T_O, H_o, W_o, T_O], and the reshape back to NCHW.  Where the printed algorithm is
inconsistent, the reading used is: the output-channel index of the kernel reshape is
k*T_O + co + j*KPG (k = output-channel tile), the convolution body's `ic`, `ocb`, `k_w` are its
loop variables c, ocv, kw, and both tile sizes must divide KPG and CPG.
"""
import numpy as np


def gspc(x, w, stride, pad, groups, T_I, T_O):
    x = np.asarray(x, dtype=np.float64)
    w = np.asarray(w, dtype=np.float64)
    N, C_in, H, W = x.shape
    C_out, CPG, KH, KW = w.shape
    KPG = C_out // groups
    assert CPG == C_in // groups and KPG % T_O == 0 and CPG % T_I == 0
    xp = np.zeros((N, C_in, H + 2 * pad, W + 2 * pad))
    xp[:, :, pad:pad + H, pad:pad + W] = x
    Hi, Wi = xp.shape[2], xp.shape[3]
    Ho = (Hi - KH) // stride + 1
    Wo = (Wi - KW) // stride + 1

    # stage 1: kernels reshaping
    Wp = np.empty((groups, KPG // T_O, CPG // T_I, KH, KW, T_I, T_O))
    for j in range(groups):
        for k in range(KPG // T_O):
            for c in range(CPG // T_I):
                for ci in range(T_I):
                    for co in range(T_O):
                        Wp[j, k, c, :, :, ci, co] = w[k * T_O + co + j * KPG, c * T_I + ci]
    # stage 2: inputs reshaping
    Xp = np.empty((groups, N, CPG // T_I, Hi, T_I, Wi))
    for j in range(groups):
        for C in range(CPG // T_I):
            for c in range(T_I):
                Xp[j, :, C, :, c, :] = xp[:, C * T_I + c + CPG * j]
    # stage 3: convolution on the packed volumes
    Yp = np.zeros((groups, N, KPG // T_O, Ho, Wo, T_O))
    for j in range(groups):
        for n in range(N):
            for occ in range(KPG // T_O):
                for oh in range(Ho):
                    for ow in range(Wo):
                        for c in range(CPG):
                            for kh in range(KH):
                                for kw in range(KW):
                                    xv = Xp[j, n, c // T_I, oh * stride + kh, c % T_I, ow * stride + kw]
                                    Yp[j, n, occ, oh, ow, :] += xv * Wp[j, occ, c // T_I, kh, kw, c % T_I, :]
    # stage 4: outputs reshaping
    Y = np.empty((N, C_out, Ho, Wo))
    for c in range(C_out):
        Y[:, c] = Yp[c // KPG, :, (c // T_O) % (KPG // T_O), :, :, c % T_O]
    return Y
