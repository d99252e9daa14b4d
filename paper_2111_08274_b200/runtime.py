"""Device memory, streams and the per-round call sequence around the C-ABI library.

PyTorch is used here for plumbing only: it owns the arena tensors and the stream.  Every step of
a round is a call into libhadfl.so.
"""
import numpy as np
import torch

from . import binding
from . import build as _build


def ensure_built():
    """Compiles libhadfl.so if its sources are newer (needs nvcc); raises if that fails."""
    return _build.build()


class Arena:
    """[N][stride] parameter and momentum tensors on one GPU plus the library handle over them."""

    def __init__(self, wl, device="cuda:0", stream=None):
        if not torch.cuda.is_available():
            raise RuntimeError("a CUDA device is required: this path has no CPU implementation")
        self.wl = wl
        self.device = torch.device(device)
        torch.cuda.set_device(self.device)
        self.stream = stream if stream is not None else torch.cuda.current_stream(self.device)
        self.stride = (wl.n_params + 31) // 32 * 32
        wdtype = torch.bfloat16 if wl.dtype == binding.DTYPE_BF16 else torch.float32
        self.w = torch.empty((wl.n_devices, self.stride), dtype=wdtype, device=self.device)
        mdtype = torch.bfloat16 if wl.m_dtype == binding.DTYPE_BF16 else torch.float32
        self.m = torch.empty((wl.n_devices, self.stride), dtype=mdtype, device=self.device)
        with torch.cuda.stream(self.stream):
            self.h = binding.Hadfl.from_workload(wl, w_ptr=self.w.data_ptr(), m_ptr=self.m.data_ptr(),
                                                 row_stride_elems=self.stride,
                                                 stream=self.stream.cuda_stream)
        if wl.sync_beta != 1.0:
            self.h.set_sync_beta(wl.sync_beta)
        self.ids = wl.device_ids()
        self.select_seed = wl.select_seed()

    def close(self):
        if self.h is not None:
            self.h.destroy()
            self.h = None

    def run_round_fused(self, r):
        """The same round as run_round through the single fused kernel (hadfl_round)."""
        wl = self.wl
        sync = bool(wl.sync_every) and (r + 1) % wl.sync_every == 0
        return self.h.round(self.ids, wl.steps_for_round(r), wl.lr, r, wl.k, self.select_seed,
                            sync_all=sync)

    def run_rounds_fused(self, first_round, n_rounds):
        """n_rounds consecutive rounds enqueued by ONE library call (hadfl_rounds)."""
        wl = self.wl
        steps = np.stack([wl.steps_for_round(first_round + i) for i in range(n_rounds)])
        return self.h.rounds(first_round, steps, wl.lr, wl.k, self.select_seed, wl.sync_every)

    def run_round(self, r, stats=True):
        """One round of the hot path as separate calls: local steps of every device, selection,
        aggregation with write-back (plus, on the workload's global-synchronisation rounds, the
        send to the unselected devices), statistics.  Returns the selected ids (draw order)."""
        wl, h = self.wl, self.h
        h.local_step(self.ids, wl.steps_for_round(r), wl.lr)
        sel = h.select(r, wl.k, self.select_seed)
        h.aggregate(sel)
        if wl.sync_every and (r + 1) % wl.sync_every == 0:
            others = np.setdiff1d(self.ids, sel).astype(np.int32)
            if wl.sync_beta == 1.0:
                h.broadcast(int(sel[0]), others)
            else:
                h.integrate(int(sel[0]), others, wl.sync_beta)
        if stats:
            h.stats_enqueue(int(sel[0]))
        return sel
