"""Helpers shared by the GPU parity tests: build both sides from the same seeded inputs."""
import numpy as np
import torch

import ssd_synth
import paper_2308_04623_b200 as ssd
from oracle import ssd_oracle, w8_oracle


class Pair:
    """One model held by the CUDA library and by the oracle, each with its own cache."""

    def __init__(self, cfg_name, seed=0, qk_gain=1.0, on_grid=False, **overrides):
        self.cfg = ssd_synth.config(cfg_name, **overrides)
        w = ssd_synth.make_weights(self.cfg, seed=seed, qk_gain=qk_gain)
        if on_grid:  # the streamed matrices moved onto the 8-bit code grid: the 8-bit library model and the oracle hold the same numbers
            w = w8_oracle.model_on_the_grid(w)
        self.weights = w
        self.oracle = ssd_oracle.Model(self.cfg, w)
        self.okv = self.oracle.new_kv()
        self.ctx = ssd.Context(self.cfg, device=0, stream=torch.cuda.current_stream().cuda_stream)
        self.ctx.load_weights(ssd_synth.bf16_bits(w) if self.cfg["dtype"] != "fp32" else w)
        self.kv = self.ctx.new_kv()
        self.V = self.cfg["vocab"]

    def prefill(self, prefix, chunk=64):
        """Prefix built with hot-path calls only on both sides (chain trees, all committed)."""
        prefix = np.asarray(prefix, dtype=np.int32)
        self.okv.prefill(prefix, chunk=chunk)
        for s in range(0, len(prefix), chunk):
            t = prefix[s:s + chunk]
            par = ssd_synth.tree_chain(len(t))
            buf = torch.empty((len(t), self.V), dtype=torch.float32, device="cuda")
            self.ctx.verify_tree(t, par, self.kv, buf.data_ptr())
            self.ctx.kv_commit(self.kv, np.arange(len(t), dtype=np.int32))
        assert len(self.kv) == len(self.okv) == len(prefix)

    def verify(self, tokens, parent):
        """Returns (gpu logits as float64 numpy, oracle logits float64)."""
        buf = torch.full((len(tokens), self.V), float("nan"), dtype=torch.float32, device="cuda")
        self.ctx.verify_tree(tokens, parent, self.kv, buf.data_ptr())
        torch.cuda.synchronize()
        want = self.okv.verify_tree(tokens, parent)
        return buf.cpu().numpy().astype(np.float64), want, buf

    def commit(self, path):
        self.ctx.kv_commit(self.kv, path)
        self.okv.commit(path)

    def close(self):
        self.kv.close()
        self.ctx.close()


def device_f32(a):
    return torch.from_numpy(np.ascontiguousarray(a, dtype=np.float32)).cuda()
