"""An independent statement of the layer built from torch CPU fp64 library routines
(matmul, silu, index_add, autograd).  It is organised expert-major with masks, unlike the
oracle's token-major loops, and its gradients come from autograd rather than from
hand-written formulas; the oracle tests compare against it."""
import torch
import torch.nn.functional as Fn


def moe_ffn_torch(x, ids, w, W_gate_up, W_down, S=0):
    """x [T,d], ids [T,k] int64, w [T,k], W_gate_up [E+S,2F,d], W_down [E+S,d,F] (all fp64)."""
    T, d = x.shape
    Ep = W_gate_up.shape[0]
    E = Ep - S
    F = W_gate_up.shape[1] // 2
    out = torch.zeros(T, d, dtype=x.dtype)
    for e in range(Ep):
        if e < E:
            tok, slot = torch.nonzero(ids == e, as_tuple=True)
            if tok.numel() == 0:
                continue
            we = w[tok, slot]
        else:
            tok = torch.arange(T)
            we = torch.ones(T, dtype=x.dtype)
        h = x[tok] @ W_gate_up[e].T
        a = Fn.silu(h[:, :F]) * h[:, F:]
        y = a @ W_down[e].T
        out = out.index_add(0, tok, y * we[:, None])
    return out
