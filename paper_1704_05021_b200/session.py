"""Buffer plumbing around the C-ABI calls: one object per worker gradient layout.

Allocates (with PyTorch) the residual, the outputs and the workspaces that gd_compress and
gd_decompress_apply need, and issues the calls.  No arithmetic happens here.
"""
from __future__ import annotations

import json
from typing import List, Optional, Sequence

import torch

from . import binding as B


class GradDropSession:
    """Worker-side state (residual) and server-side shards for one flat gradient layout."""

    def __init__(self, layer_off: Sequence[int], shard_off: Sequence[int], drop_ppm: int,
                 scope_mode: int = B.GD_SCOPE_GLOBAL, value_mode: int = B.GD_VALUES_FP32, flags: int = 0,
                 device="cuda:0", layer_cols: Optional[Sequence[int]] = None):
        self.device = torch.device(device)
        if self.device.type != "cuda":
            raise RuntimeError("GradDropSession needs a CUDA device: the library has no CPU path")
        self.layer_off = [int(x) for x in layer_off]
        self.shard_off = [int(x) for x in shard_off]
        self.n = self.layer_off[-1]
        self.n_layers = len(self.layer_off) - 1
        self.n_shards = len(self.shard_off) - 1
        self.drop_ppm, self.scope_mode, self.value_mode, self.flags = drop_ppm, scope_mode, value_mode, flags
        self.layer_cols = [int(c) for c in layer_cols] if value_mode == B.GD_VALUES_COLUMN_MEANS else None
        self.n_pairs = B.gd_means_pairs(self.n_layers, self.layer_cols, value_mode)
        self.n_scopes = 1 if scope_mode == B.GD_SCOPE_GLOBAL else self.n_layers
        self.sampled = bool(flags & B.GD_FLAG_SAMPLED_THRESHOLD)
        # exact modes: the survivor count is known; sampled-threshold mode: the capacity of the outputs
        self.k_total = (B.gd_sampled_capacity(self.layer_off, scope_mode, drop_ppm) if self.sampled
                        else B.gd_total_kept(self.layer_off, scope_mode, drop_ppm))
        dev = self.device
        self.residual = torch.empty(self.n, dtype=torch.float32, device=dev)
        self.out_idx = torch.zeros(max(self.k_total, 1), dtype=torch.int32, device=dev)
        self.out_val = torch.zeros(max(self.k_total, 1), dtype=torch.float32, device=dev)
        self.out_shard_cnt_off = torch.zeros(self.n_shards + 1, dtype=torch.int32, device=dev)
        self.out_tau = torch.zeros(self.n_scopes, dtype=torch.int32, device=dev)
        self.out_means = torch.zeros(max(self.n_pairs, 1), 2, dtype=torch.float32, device=dev)
        ws_bytes = B.gd_workspace_bytes(self.layer_off, self.n_shards, scope_mode, drop_ppm, self.layer_cols)
        self.workspace = torch.empty(ws_bytes, dtype=torch.uint8, device=dev)
        aws = B.gd_apply_workspace_bytes(self.n_shards, self.n_layers)
        self.apply_workspace = torch.empty(aws, dtype=torch.uint8, device=dev)
        self._compress_call: Optional[B.CompressCall] = None
        self._apply_call: Optional[B.ApplyCall] = None
        self._apply_params = None                     # the list the cached argument block was built from
        self.reset()

    def reset(self, stream=None) -> None:
        B.gd_residual_reset(self.residual, stream)

    def compress_call(self, grad: torch.Tensor) -> B.CompressCall:
        assert grad.is_cuda and grad.dtype == torch.float32 and grad.numel() == self.n and grad.is_contiguous()
        if self._compress_call is None:
            self._compress_call = B.CompressCall(
                grad, self.residual, self.layer_off, self.shard_off, self.drop_ppm, self.scope_mode, self.value_mode,
                self.out_idx, self.out_val, self.out_shard_cnt_off, self.out_tau, self.out_means, self.workspace,
                self.flags, layer_cols=self.layer_cols)
        else:
            self._compress_call.set_grad(grad)
        return self._compress_call

    def compress(self, grad: torch.Tensor, stream=None) -> None:
        B.gd_compress(self.compress_call(grad), stream)

    def compress_delta(self, params: torch.Tensor, last_pulled: torch.Tensor, stream=None) -> None:
        """Server side of a pull: GradDrop of params - last_pulled; the survivors are added to last_pulled."""
        assert last_pulled.is_cuda and last_pulled.dtype == torch.float32 and last_pulled.numel() == self.n
        call = B.CompressCall(params, self.residual, self.layer_off, self.shard_off, self.drop_ppm, self.scope_mode,
                              self.value_mode, self.out_idx, self.out_val, self.out_shard_cnt_off, self.out_tau,
                              self.out_means, self.workspace, self.flags, delta_base=last_pulled)
        B.gd_compress(call, stream)

    def push(self) -> dict:
        """The last compress call's output as a push record for ApplyCall."""
        p = {"idx": self.out_idx, "shard_cnt_off": self.out_shard_cnt_off}
        if self.value_mode != B.GD_VALUES_FP32:
            p["means"] = self.out_means
        else:
            p["val"] = self.out_val
        return p

    def apply_call(self, params: List[torch.Tensor], alpha: float = 1.0, pushes=None, flags: int = 0) -> B.ApplyCall:
        pushes = [self.push()] if pushes is None else pushes
        lo = self.layer_off if self.value_mode != B.GD_VALUES_FP32 else None
        return B.ApplyCall(params, self.shard_off, pushes, self.value_mode, alpha, self.apply_workspace, lo,
                           self.layer_cols, flags)

    def apply(self, params: List[torch.Tensor], alpha: float = 1.0, stream=None) -> None:
        if self._apply_call is None or self._apply_params is not params:
            self._apply_call = self.apply_call(params, alpha)
            self._apply_params = params
        self._apply_call.args.alpha = float(alpha)       # (the cached argument block may carry another call's alpha)
        B.gd_decompress_apply(self._apply_call, stream)

    def shard_views(self, flat_params: torch.Tensor) -> List[torch.Tensor]:
        return [flat_params[self.shard_off[j]:self.shard_off[j + 1]] for j in range(self.n_shards)]

    def kept(self) -> int:
        """Survivors of the last compress call (a device read in sampled-threshold mode)."""
        return int(self.out_shard_cnt_off[-1].item()) if self.sampled else self.k_total

    def status(self) -> int:
        return B.gd_status(self.workspace)

    def stats(self) -> dict:
        return B.gd_get_stats(self.workspace)

    def log_step(self, fh, step: int, **extra) -> dict:
        """Appends one JSON line about the last compress call to the open text file `fh` and returns it: the step
        number, the call's status and counters (gd_get_stats), the survivors per shard and the scopes' threshold keys.
        Waits for the stream (the figures are read from the device), so it is for logs, not for the timed path."""
        off = self.out_shard_cnt_off.cpu().tolist()
        rec = {"step": int(step), **self.stats(),
               "kept_per_shard": [int(off[j + 1] - off[j]) for j in range(self.n_shards)],
               "tau_keys": [int(x) & 0xFFFFFFFF for x in self.out_tau.cpu().tolist()], **extra}
        fh.write(json.dumps(rec) + "\n")
        return rec
