"""GPU-side test plumbing: numpy rank buffers in, numpy receive buffers out, through the C ABI."""
import numpy as np
import torch

from paper_2608_00358_b200.runtime import DeviceCollective

GUARD = 256
SENTINEL = 0xA5


def run_plan(plan, X, iters=1, misalign=0, stream=None):
    """Execute `plan` on device copies of X (list of numpy arrays). Receive buffers are pre-filled with a
    sentinel and wrapped in guard bands that must survive. Returns per-rank uint8 numpy arrays."""
    info = plan.info()
    R = info.R
    dev = "cuda"
    send_t, recv_t, sp, rp = [], [], [], []
    for r in range(R):
        s, v = plan.extents(r)
        assert X[r].nbytes >= s
        t = torch.full((max(s, 16) + 2 * GUARD + 32,), SENTINEL, dtype=torch.uint8, device=dev)
        off = GUARD + misalign
        if s:
            t[off:off + s] = torch.from_numpy(X[r].view(np.uint8).reshape(-1)[:s].copy()).to(dev)
        send_t.append(t)
        sp.append(t.data_ptr() + off)
        u = torch.full((max(v, 16) + 2 * GUARD + 32,), SENTINEL, dtype=torch.uint8, device=dev)
        recv_t.append(u)
        rp.append(u.data_ptr() + off)
    dc = DeviceCollective(plan, stream=stream)
    dc.set_buffers(sp, rp, keep=(send_t, recv_t))
    for _ in range(iters):
        dc.execute()
    dc.check()
    out = []
    for r in range(R):
        s, v = plan.extents(r)
        h = recv_t[r].cpu().numpy()
        off = GUARD + misalign
        assert np.all(h[:off] == SENTINEL) and np.all(h[off + v:] == SENTINEL), "guard band of rank %d overwritten" % r
        hs = send_t[r].cpu().numpy()
        assert np.array_equal(hs[off:off + s], X[r].view(np.uint8).reshape(-1)[:s]), "send buffer of rank %d modified" % r
        out.append(h[off:off + v].copy())
    return out
