"""Builds a synthetic weight pass on the device: seeded codes, scales,
activations and tails for a list of matrices, packed for the GEMV kernels.

Input generation and argument marshalling only; all arithmetic of the method
runs in the CUDA library.
"""
from typing import List, Optional

import numpy as np
import torch

from . import shapes, synth, tetra


class DevicePass:
    """Device-resident inputs and outputs of a list of products.

    All activations live in one buffer (x_all) and all results in another
    (y_all), so a whole pass moves between host and device in one copy each way.
    """

    def __init__(self, matrices: List[shapes.Matrix], seed: int = 0, tail_mode: bool = True,
                 gain=None, device="cuda", keep_file_codes: bool = False, stream_base: int = 0):
        self.matrices = list(matrices)
        self.tail_mode = tail_mode
        self.seed = seed
        self.device = device
        self.gain = np.asarray(synth.DEFAULT_GAIN if gain is None else gain, dtype=np.float32)
        self.table = tetra.tetra_build_table(self.gain, device=device)
        xoff, yoff = [], []
        xn = yn = 0
        for m in self.matrices:
            xoff.append(xn)
            yoff.append(yn)
            xn += -(-m.K // 8) * 8          # keep every x 16-byte aligned
            yn += -(-m.N // 4) * 4
        self.x_host = torch.zeros(xn, dtype=torch.float16).pin_memory() if device != "cpu" else None
        self.x_all = torch.zeros(xn, dtype=torch.float16, device=device)
        self.y_all = torch.zeros(yn, dtype=torch.float32, device=device)
        self.y_host = torch.zeros(yn, dtype=torch.float32).pin_memory() if device != "cpu" else None
        self.items = []
        self.algorithmic_bytes = 0
        self.code_bytes = 0
        self.blocks = 0
        for i, m in enumerate(self.matrices):
            stream = stream_base + i
            B = m.blocks if tail_mode else m.blocks_padded
            ntail = m.ntail if tail_mode else 0
            file_codes = synth.codes_torch(seed, stream, m.N, B, device=device)
            packed = tetra.tetra_pack_codes(file_codes, self.table, m.N, B)
            sigma = synth.row_scales(seed, stream, m.N)
            x = synth.activations(seed, stream, m.K)[0]
            tail = synth.tails(seed, stream, sigma, ntail) if ntail else None
            self.x_host[xoff[i]:xoff[i] + m.K] = torch.from_numpy(x)
            it = dict(name=m.name, N=m.N, K=m.K, B=B, ntail=ntail, stream=stream,
                      codes=packed,
                      codes_file=file_codes if keep_file_codes else None,
                      row_scales=torch.from_numpy(sigma).to(device),
                      x=self.x_all[xoff[i]:xoff[i] + m.K],
                      tail=torch.from_numpy(tail).to(device) if tail is not None else None,
                      y=self.y_all[yoff[i]:yoff[i] + m.N],
                      xoff=xoff[i], yoff=yoff[i])
            self.items.append(it)
            nbytes = packed.numel() + m.N * 4 + m.K * 2 + m.N * 4 + m.N * ntail * 2
            it["bytes"] = nbytes
            self.algorithmic_bytes += nbytes
            self.code_bytes += packed.numel()
            self.blocks += m.N * B
        self.x_all.copy_(self.x_host)
        torch.cuda.synchronize()
        self.problems = tetra.make_problems(self.items)
        self.workspace = torch.empty(max(16, tetra.tetra_grouped_workspace_bytes(self.problems)),
                                     dtype=torch.uint8, device=device)
        tetra.tetra_gemv_grouped_plan(self.problems, self.workspace)
        torch.cuda.synchronize()

    # ---- the three ways to run the pass ---------------------------------
    def run_grouped(self, stream=None):
        tetra.tetra_gemv_grouped_run(self.workspace, self.table, stream=stream)

    def run_per_matrix(self, stream=None):
        for it in self.items:
            tetra.tetra_gemv_tail(it["codes"], it["row_scales"], self.table, it["x"], it["y"], it["N"], it["K"], 1,
                                  it["tail"], stream=stream)

    def run_paper_design(self, stream=None):
        for it in self.items:
            tetra.tetra_gemv_paper_design(it["codes_file"], 6 * it["B"], it["row_scales"], self.table, it["x"],
                                          it["y"], it["N"], it["K"], 1, it["tail"], stream=stream)

    def run_grouped_hostio(self, stream=None):
        tetra.tetra_gemv_grouped_hostio(self.workspace, self.table, self.x_host, self.x_all,
                                        self.y_host, self.y_all, stream=stream)

    def plan_mapped_results(self):
        """A second plan of the same list whose results go straight to pinned host memory (y_mapped)."""
        self.y_mapped = torch.zeros_like(self.y_host).pin_memory()
        items = []
        for it in self.items:
            j = dict(it)
            j["y"] = self.y_mapped[it["yoff"]:it["yoff"] + it["N"]]
            items.append(j)
        self.problems_mapped = tetra.make_problems(items)
        self.workspace_mapped = torch.empty(max(16, tetra.tetra_grouped_workspace_bytes(self.problems_mapped)),
                                            dtype=torch.uint8, device=self.device)
        tetra.tetra_gemv_grouped_plan(self.problems_mapped, self.workspace_mapped)
        torch.cuda.synchronize()

    def run_grouped_mapped(self, stream=None):
        tetra.tetra_gemv_grouped_hostio(self.workspace_mapped, self.table, self.x_host, self.x_all, stream=stream)

    # ---- host copies for the checker ---------------------------------------
    def host_inputs(self, index: int, rows: Optional[np.ndarray] = None):
        """File-order codes (regenerated from the seed), scales, x and tail of matrix
        `index` on the host, all rows or the listed ones."""
        it = self.items[index]
        codes = synth.codes(self.seed, it["stream"], it["N"], it["B"]) if rows is None else None
        if rows is not None:
            rows = np.asarray(rows)
            sel = [synth.words_to_bytes(synth.words(self.seed, it["stream"], it["B"], int(r) * it["B"]))
                   for r in rows]
            codes = np.stack(sel).reshape(len(rows), it["B"], 6)
        sigma = synth.row_scales(self.seed, it["stream"], it["N"])
        x = synth.activations(self.seed, it["stream"], it["K"])
        tail = synth.tails(self.seed, it["stream"], sigma, it["ntail"]) if it["ntail"] else None
        if rows is not None:
            sigma = sigma[rows]
            tail = tail[rows] if tail is not None else None
        return dict(N=len(sigma), K=it["K"], B=it["B"], ntail=it["ntail"], codes=codes, sigma=sigma, x=x, tail=tail)
