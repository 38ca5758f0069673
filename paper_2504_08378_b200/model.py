"""Host-side convenience around the model / state entry points of libafx.

Uploads one layer's weights (torch is used for device memory only), fills the C
descriptors, and exposes the buffers inside the state blob as torch views.  All
computation happens in the library's kernels.
"""
from __future__ import annotations

import numpy as np
import torch

from . import afx, synth

_TORCH_16 = {"f16": torch.float16, "bf16": torch.bfloat16}


def to_device_bits(a) -> torch.Tensor:
    if isinstance(a, torch.Tensor):
        return a.cuda().contiguous()
    a = np.ascontiguousarray(a)
    if a.dtype == np.uint16:
        return torch.from_numpy(a.view(np.int16)).cuda()
    return torch.from_numpy(a).cuda()


class DecoderModel:
    """Llama-shaped stack with sparse operators.

    layers: list of dicts with numpy bit-pattern weights ``w_qkv, w_o, w_gate, w_up, w_down``,
    fp32 gains ``g_attn, g_mlp``, optional ``k`` / ``tau`` (length-4 sequences indexed by
    afx.OP_*), optional caches ``k_cache, v_cache`` ([T][max_seq][n_kv][128] uint16).
    """

    def __init__(self, dtype: str, hidden: int, n_heads: int, n_kv_heads: int, mlp: int, max_seq: int,
                 layers, T: int = 1, select_mode: int = afx.MODE_TOPK, xl_depth: int = 0,
                 xl_mode: int = afx.XL_OFF, eps: float = 1e-5, theta: float = 10000.0, head_dim: int = 128):
        self.dtype, self.hidden, self.n_heads, self.n_kv_heads = dtype, hidden, n_heads, n_kv_heads
        self.mlp, self.max_seq, self.T, self.head_dim = mlp, max_seq, T, head_dim
        self.n_qkv = (n_heads + 2 * n_kv_heads) * head_dim
        self.K_op = [hidden, n_heads * head_dim, hidden, mlp]
        self._keep = []
        descs = []
        self.k_cache, self.v_cache, self.q4 = [], [], []
        for L in layers:
            d = afx.LayerDesc()
            # 16-bit weights may be absent when the layer is only stepped over 4-bit rows ("q4")
            w_gu = L.get("w_gu")
            if w_gu is None and L.get("w_gate") is not None:
                w_gu = synth.interleave_gate_up(L["w_gate"], L["w_up"])
            dev = lambda w: None if w is None else to_device_bits(w)
            tens = dict(w_qkv=dev(L.get("w_qkv")), w_o=dev(L.get("w_o")), w_gu=dev(w_gu), w_down=dev(L.get("w_down")),
                        g_attn=to_device_bits(L["g_attn"]).float(), g_mlp=to_device_bits(L["g_mlp"]).float())
            q4 = None
            if L.get("q4") is not None:  # per operator a uint8 CUDA tensor [K_op][row bytes] or None
                q4 = afx.Q4Layer()
                for op, rows in enumerate(L["q4"]):
                    q4.wq[op] = None if rows is None else rows.data_ptr()
                    q4.ldq_bytes[op] = 0 if rows is None else rows.shape[1]
                tens["q4"] = L["q4"]
            self.q4.append(q4)
            if "k_cache" in L:
                kc, vc = to_device_bits(L["k_cache"]), to_device_bits(L["v_cache"])
            else:
                kc = torch.zeros((T, max_seq, n_kv_heads, head_dim), dtype=torch.int16, device="cuda")
                vc = torch.zeros_like(kc)
            self.k_cache.append(kc)
            self.v_cache.append(vc)
            tens["k_cache"], tens["v_cache"] = kc, vc
            for name, t in tens.items():
                if name != "q4":
                    setattr(d, name, None if t is None else t.data_ptr())
            for op in range(4):
                d.k[op] = int(L.get("k", [0, 0, 0, 0])[op])
                d.tau[op] = float(L.get("tau", [0.0, 0.0, 0.0, 0.0])[op])
            self._keep.append(tens)
            descs.append(d)
        md = afx.ModelDesc(dtype=afx.DTYPES[dtype], n_layers=len(layers), hidden=hidden, n_heads=n_heads,
                           n_kv_heads=n_kv_heads, head_dim=head_dim, mlp=mlp, max_seq=max_seq, rms_eps=eps,
                           rope_theta=theta, select_mode=select_mode, xl_depth=xl_depth, xl_mode=xl_mode)
        self.n_layers = len(layers)
        self.handle = afx.afx_model_create(md, descs)
        nbytes = afx.afx_state_bytes(self.handle, T)
        raw = torch.empty(nbytes + 256, dtype=torch.uint8, device="cuda")
        off = (-raw.data_ptr()) % 256
        self.blob = raw[off:off + nbytes]
        self.state = afx.afx_state_create(self.handle, T, self.blob, nbytes)
        torch.cuda.synchronize()

    def close(self):
        if self.state:
            afx.afx_state_destroy(self.state)
            self.state = None
        if self.handle:
            afx.afx_model_destroy(self.handle)
            self.handle = None

    def __del__(self):
        try:
            self.close()
        except Exception:
            pass

    def _view(self, which: int, op: int, tdtype, shape):
        ptr, n = afx.afx_state_buffer(self.state, which, op)
        off = ptr - self.blob.data_ptr()
        return self.blob[off:off + n].view(tdtype).view(*shape)

    @property
    def h(self) -> torch.Tensor:
        return self._view(afx.BUF_H, 0, torch.float32, (self.T, self.hidden))

    @property
    def qkv(self) -> torch.Tensor:
        return self._view(afx.BUF_QKV, 0, torch.float32, (self.T, self.n_qkv))

    def bits(self, which: int, op: int = 0) -> torch.Tensor:
        """int16 view of a 16-bit buffer (ATTN, HM, XNORM)."""
        width = {afx.BUF_ATTN: self.n_heads * self.head_dim, afx.BUF_HM: self.mlp,
                 afx.BUF_XNORM: self.hidden}[which]
        return self._view(which, op, torch.int16, (self.T, width))

    def idx(self, op: int) -> torch.Tensor:
        return self._view(afx.BUF_IDX, op, torch.int32, (self.K_op[op],))

    def miss(self, op: int) -> torch.Tensor:
        return self._view(afx.BUF_MISS, op, torch.int32, (self.K_op[op],))

    @property
    def stats(self) -> torch.Tensor:
        return self._view(afx.BUF_STATS, 0, torch.int32, (self.n_layers, 4, 4))

    @property
    def hints(self) -> torch.Tensor:
        return self._view(afx.BUF_HINTS, 0, torch.int32, (self.n_layers, 4, afx.MAX_T))

    def layer_step(self, layer: int, pos: int, stream=None):
        afx.afx_layer_step(self.handle, layer, self.state, pos, stream)

    def layer_kernel(self, layer: int, pos: int, which: int, stream=None):
        afx.afx_layer_kernel(self.handle, layer, self.state, pos, which, stream)

    def decode_step(self, pos: int, stream=None):
        for layer in range(self.n_layers):
            afx.afx_layer_step(self.handle, layer, self.state, pos, stream)

    def layer_step_q4(self, layer: int, pos: int, stream=None, dev_status=None):
        afx.afx_layer_step_q4(self.handle, layer, self.state, pos, self.q4[layer], stream, dev_status)

    def decode_step_q4(self, pos: int, stream=None, dev_status=None):
        for layer in range(self.n_layers):
            afx.afx_layer_step_q4(self.handle, layer, self.state, pos, self.q4[layer], stream, dev_status)

    def mlp_block(self, layer: int, x: torch.Tensor, y: torch.Tensor, stream=None):
        afx.afx_mlp_block(self.handle, layer, self.state, x, y, stream)
