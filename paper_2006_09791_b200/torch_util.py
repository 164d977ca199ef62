"""Device-memory plumbing for callers that hold their tensors in PyTorch (no arithmetic here)."""
from __future__ import annotations

from . import gconv


def attach_workspace(desc, device):
    """Allocates the workspace the descriptor's variant needs (gconv_workspace_bytes, zero for most layers) as a
    torch tensor on `device` and attaches it with gconv_desc_set_workspace.  Returns the tensor -- the caller keeps it
    alive as long as the descriptor is used -- or None when no workspace is needed."""
    import torch

    need = gconv.gconv_workspace_bytes(desc)
    if need == 0:
        return None
    ws = torch.empty((need + 3) // 4, dtype=torch.float32, device=device)
    gconv.gconv_desc_set_workspace(desc, ws, ws.numel() * 4)
    return ws
