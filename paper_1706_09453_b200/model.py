"""Put a synthetic network on the GPU: upload the real-valued parameters, binarise and pack
the weights (Eq. 3) and fold the hidden layers' affine + Sign into thresholds -- all with the
library's own kernels -- and describe it as a ``bnn_model`` for ``bnn_forward``."""
from __future__ import annotations

import numpy as np
import torch

from . import binding as B
from . import workloads as wl


def to_dev(a: np.ndarray, device="cuda:0") -> torch.Tensor:
    if a.dtype == np.uint32:
        a = a.view(np.int32)
    return torch.from_numpy(np.ascontiguousarray(a)).to(device)


def packed_empty(rows: int, k: int, device="cuda:0") -> torch.Tensor:
    return torch.empty((rows, B.packed_pitch(k)), dtype=torch.int32, device=device)


def words_to_numpy(t: torch.Tensor, k: int) -> np.ndarray:
    """Packed device tensor -> numpy uint32 [rows][ceil(k/32)] (pitch words dropped)."""
    return t.cpu().numpy().view(np.uint32)[:, :(k + 31) // 32].copy()


class DeviceNet:
    def __init__(self, net: wl.Model, sign_mode=B.SIGN_ZERO_POS, device="cuda:0", prepare_xnor=True,
                 act_values=B.VALUES_PM1, splice=(0, 0), log_prior=None):
        cfg = net.cfg
        self.cfg, self.sign_mode, self.device = cfg, sign_mode, device
        self.Wp, self.scale, self.shift, self.thr, self.flip, self.Wimg = [], [], [], [], [], []
        layers = []
        binary_act = cfg.act == wl.ACT_SIGN
        mixed = getattr(cfg, "mixed", False)
        self.W0 = self.W0_prepared = None
        for l, w in enumerate(net.W):
            n, k = w.shape
            wd = to_dev(w, device)
            if mixed and l == 0:
                # real-valued Sigmoid layer: the weights as they are, prepared for the tensor cores
                self.W0 = wd
                self.W0_prepared = torch.empty(B.bnn_output_prepared_bytes(n, k), dtype=torch.uint8, device=device)
                B.bnn_output_prepare(wd, self.W0_prepared)
                sh = to_dev(net.shift[l], device)
                self.Wp.append(None); self.scale.append(None); self.shift.append(sh)
                self.thr.append(None); self.flip.append(None)
                layers.append(dict(kind=B.LAYER_REAL, K=k, N=n, W=wd, W_prepared=self.W0_prepared, shift=sh,
                                   act=B.ACT_SIGMOID))
                continue
            wp = packed_empty(n, k, device)
            B.bnn_pack_weights(wd, wp, sign_mode)
            del wd
            sc, sh = to_dev(net.scale[l], device), to_dev(net.shift[l], device)
            self.Wp.append(wp); self.scale.append(sc); self.shift.append(sh)
            first_binary = l == (1 if mixed else 0)
            if first_binary or not binary_act:
                layers.append(dict(kind=B.LAYER_SIGNW, K=k, N=n, Wp=wp, scale=sc, shift=sh,
                                   act=B.ACT_SIGN_PACK if binary_act else B.ACT_HARDTANH))
                self.thr.append(None); self.flip.append(None)
            else:
                last_sigmoid = mixed and l == len(net.W) - 1
                thr = torch.empty(n, dtype=torch.int32, device=device)
                flip = torch.empty((n + 31) // 32, dtype=torch.int32, device=device)
                B.bnn_fold_thresholds(sc, sh, n, k, thr, flip, sign_mode)
                self.thr.append(thr); self.flip.append(flip)
                img = None
                if prepare_xnor:   # widened image of the weights for the tensor cores (built once)
                    img = torch.empty(B.bnn_xnor_prepared_bytes(n, k), dtype=torch.uint8, device=device)
                    B.bnn_xnor_prepare(wp, k, img)
                self.Wimg.append(img)
                layers.append(dict(kind=B.LAYER_XNOR, K=k, N=n, Wp=wp, thr=thr, flip=flip, W_prepared=img,
                                   scale=sc, shift=sh,
                                   act=B.ACT_SIGMOID if last_sigmoid else B.ACT_SIGN_PACK))
        self.Wout, self.bout = to_dev(net.Wout, device), to_dev(net.bout, device)
        self.Wout_prepared = torch.empty(B.bnn_output_prepared_bytes(cfg.classes, cfg.hidden),
                                         dtype=torch.uint8, device=device)
        B.bnn_output_prepare(self.Wout, self.Wout_prepared)
        layers.append(dict(kind=B.LAYER_REAL_OUT, K=cfg.hidden, N=cfg.classes, W=self.Wout,
                           W_prepared=self.Wout_prepared, shift=self.bout))
        self.log_prior = to_dev(log_prior, device) if log_prior is not None else None
        self.desc = B.ModelDesc(layers, sign_mode, act_values, splice, self.log_prior)
        self._ws = None

    def workspace(self, M: int) -> torch.Tensor:
        need = self.desc.workspace_bytes(M)
        if self._ws is None or self._ws.numel() < need:
            self._ws = torch.empty(need, dtype=torch.uint8, device=self.device)
        return self._ws

    def forward(self, X: torch.Tensor, logp: torch.Tensor | None = None, layer_out=None):
        M = X.shape[0]
        if logp is None:
            logp = torch.empty((M, self.cfg.classes), dtype=torch.float32, device=self.device)
        return B.bnn_forward(self.desc, X, logp, self.workspace(M), layer_out)

    def layer_out_buffers(self, M: int):
        """One tensor per hidden layer, shaped as bnn_forward writes it."""
        outs = []
        for d in self.desc.layers[:-1]:
            if d["act"] == B.ACT_SIGN_PACK:
                outs.append(packed_empty(M, d["N"], self.device))
            else:
                outs.append(torch.empty((M, d["N"]), dtype=torch.float32, device=self.device))
        return outs
