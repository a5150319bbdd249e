"""Device-resident 4-bit linears of a Llama-2-7B decoder stack (the OpenVLA backbone) and the
descriptor list that runs one pass over them through the C ABI.

Setup (draw weights on the host, quantise and pack them on the device with the library's own
quantiser) happens once; ``run()`` / ``run_host()`` only enqueue the linears.  The inputs of the
linears are independent vectors (attention, norms and activations are not part of the linear path),
the calls stay in stream order.
"""
from __future__ import annotations

import ctypes as C
from concurrent.futures import ThreadPoolExecutor
import os

import numpy as np
import torch

from . import _lib, api, workloads as wl


class QuantisedLinears:
    def __init__(self, cfg: int = 1, M: int = 1, n_layers: int = wl.N_LAYERS, layout: int = api.LAYOUT_STREAM128,
                 deps: str = "none",
                 outliers: bool = True, device: str = "cuda", keep_host_rows: dict | None = None,
                 host_threads: int | None = None, bits: int = 4):
        if bits == 8:
            layout = api.LAYOUT_CANONICAL   # 8-bit codes are one byte each, row-major
        self.M, self.layout, self.device, self.bits = M, layout, device, bits
        self.lib = _lib.load()
        self.specs = [s for s in wl.llama_linear_ids() if s[0] < n_layers]
        self.G = wl.GROUP_SIZE
        self.kept = {}          # linear index -> (row ids, fp32 rows) for oracle sampling
        self.packed, self.scales, self.zeros = [], [], []
        threads = host_threads or max(1, min(16, (os.cpu_count() or 2) - 1))

        def draw(i):
            _, _, N, K, tw, _ = self.specs[i]
            return wl.llama_weight(cfg, tw, N, K, outliers)

        with ThreadPoolExecutor(max_workers=threads) as pool:
            window = threads + 2
            futs = {i: pool.submit(draw, i) for i in range(min(window, len(self.specs)))}
            for i in range(len(self.specs)):
                w = futs.pop(i).result()
                nxt = i + window
                if nxt < len(self.specs):
                    futs[nxt] = pool.submit(draw, nxt)
                if keep_host_rows and i in keep_host_rows:
                    rows = np.asarray(keep_host_rows[i])
                    self.kept[i] = (rows, w[rows].copy())
                wd = torch.from_numpy(w).to(device)
                codes, s, z = api.quantize_rtn_w8(wd, self.G) if bits == 8 else api.quantize_rtn_w4(wd, self.G)
                if bits == 8:
                    self.packed.append(codes)
                elif layout == api.LAYOUT_STREAM128:
                    self.packed.append(api.pack_stream128_w4(codes, s, z, self.G))
                else:
                    self.packed.append(api.pack_w4(codes, layout))
                self.scales.append(s)
                self.zeros.append(z)
                del wd, codes, w

        # activations: one independent bf16 vector block per linear, all in one buffer (and one for y)
        self.x_off, self.y_off = [], []
        xo = yo = 0
        for (_, _, N, K, _, _) in self.specs:
            self.x_off.append(xo)
            self.y_off.append(yo)
            xo += M * K
            yo += M * N
        self.x_elems, self.y_elems = xo, yo
        x_bits = np.empty(xo, dtype=np.uint16)
        for i, (_, _, N, K, _, tx) in enumerate(self.specs):
            x_bits[self.x_off[i]:self.x_off[i] + M * K] = wl.normal_activations_bf16(cfg, tx, M, K).reshape(-1)
        self.x_bits = x_bits
        self.x_host = torch.from_numpy(x_bits.view(np.int16)).view(torch.bfloat16).pin_memory()
        self.y_host = torch.empty(yo, dtype=torch.bfloat16).pin_memory()
        self.x_dev = self.x_host.to(device)
        self.y_dev = torch.zeros(yo, dtype=torch.bfloat16, device=device)

        if bits == 8:
            ws_bytes = max(int(self.lib.qil_linear_w8a16_workspace_size(M, N, K, self.G)) for (_, _, N, K, _, _) in self.specs)
        else:
            ws_bytes = max(api.linear_w4a16_workspace_size(M, N, K, self.G) for (_, _, N, K, _, _) in self.specs)
        self.ws = api.new_workspace(ws_bytes, device)
        self.ws_bytes = self.ws.numel()

        self.descs = (_lib.LinearDesc * len(self.specs))()
        for i, (_, _, N, K, _, _) in enumerate(self.specs):
            d = self.descs[i]
            d.x = self.x_dev.data_ptr() + 2 * self.x_off[i]
            d.qweight = self.packed[i].data_ptr()
            d.scales = self.scales[i].data_ptr()
            d.zeros = self.zeros[i].data_ptr()
            d.y = self.y_dev.data_ptr() + 2 * self.y_off[i]
            d.M, d.N, d.K, d.group_size, d.layout = M, N, K, self.G, layout
        self.set_deps(deps)

    def set_deps(self, deps: str) -> None:
        """Rewrites the ordering flags of the descriptor list (see _dep_flag)."""
        for i in range(len(self.specs)):
            self.descs[i].flags = self._dep_flag(i, deps)

    def _dep_flag(self, i: int, deps: str) -> int:
        """Which entries wait for all earlier ones.  "none": no entry (every linear reads its own input vector,
        none reads another linear's output: the GEMV throughput).  "layer": the order a decoder layer imposes
        (q after the previous layer's down, o after attention, gate after o, down after gate/up; k, v and up
        start with q / gate), as if each output fed the next input directly.  "all": every entry."""
        if deps == "all":
            return api.DEP_PREVIOUS if i > 0 else 0
        if deps == "none":
            return 0
        name = self.specs[i][1]
        return api.DEP_PREVIOUS if (name in ("q", "o", "gate", "down") and i > 0) else 0

    # ---- sizes -------------------------------------------------------------------------------
    @property
    def count(self) -> int:
        return len(self.specs)

    def weight_bytes(self) -> int:
        """Algorithmic weight-side bytes of one pass: packed codes + fp16 scales + fp16 zeros."""
        return sum(N * K * self.bits // 8 + 4 * N * (K // self.G) for (_, _, N, K, _, _) in self.specs)

    def algorithmic_bytes(self) -> int:
        """weight_bytes + activations read + outputs written (bf16)."""
        return self.weight_bytes() + 2 * self.x_elems + 2 * self.y_elems

    # ---- running -----------------------------------------------------------------------------
    def run(self, stream=None) -> None:
        """One pass over all linears, activations already on the device."""
        s = torch.cuda.current_stream() if stream is None else stream
        fn = self.lib.qil_linear_w8a16_batch if self.bits == 8 else self.lib.qil_linear_w4a16_batch
        api._check(fn(self.descs, self.count, C.c_void_p(self.ws.data_ptr()), self.ws_bytes, C.c_void_p(s.cuda_stream)))

    def run_host(self, stream=None) -> None:
        """One pass with activations in (pinned) host memory: H2D copy, linears, D2H copy."""
        s = torch.cuda.current_stream() if stream is None else stream
        api._check(self.lib.qil_linear_w4a16_batch_host(
            self.descs, self.count, C.c_void_p(self.x_host.data_ptr()), C.c_void_p(self.x_dev.data_ptr()),
            2 * self.x_elems, C.c_void_p(self.y_host.data_ptr()), C.c_void_p(self.y_dev.data_ptr()),
            2 * self.y_elems, C.c_void_p(self.ws.data_ptr()), self.ws_bytes, C.c_void_p(s.cuda_stream)))

    def output(self, i: int) -> torch.Tensor:
        _, _, N, _, _, _ = self.specs[i]
        return self.y_dev[self.y_off[i]:self.y_off[i] + self.M * N].view(self.M, N)

    def input_bits(self, i: int) -> np.ndarray:
        _, _, _, K, _, _ = self.specs[i]
        return self.x_bits[self.x_off[i]:self.x_off[i] + self.M * K].reshape(self.M, K)
