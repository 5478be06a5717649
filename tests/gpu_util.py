"""Helpers shared by the GPU parity tests: move a seeded batch to the device, call the C ABI
through the Python binding, and measure the error against the fp64 oracle."""
import numpy as np
import torch

from paper_2608_22788_b200 import api

MAX_ABS_TOL = 1e-2     # bf16 attention outputs vs the unrounded fp64 oracle
REL_L2_TOL = 2e-3


def bf16_tensor(bits: np.ndarray, device="cuda") -> torch.Tensor:
    t = torch.from_numpy(np.ascontiguousarray(bits).view(np.int16))
    return t.to(device).view(torch.bfloat16)


def bf16_to_f64(t: torch.Tensor) -> np.ndarray:
    bits = t.detach().contiguous().view(torch.int16).cpu().numpy().view(np.uint16)
    return (bits.astype(np.uint32) << np.uint32(16)).view(np.float32).astype(np.float64)


def geometry(b) -> api.AttnGeometry:
    return api.AttnGeometry(b.num_seqs, b.q_len, b.num_q_heads, b.num_kv_heads, b.head_dim, b.page_size,
                            b.num_pages, b.max_pages_per_seq, b.kv_page_stride, b.kv_token_stride,
                            b.kv_head_stride, b.scale)


class DeviceBatch:
    def __init__(self, b):
        self.b = b
        self.geom = geometry(b)
        self.q = bf16_tensor(b.q)
        self.k = bf16_tensor(b.k_pool)
        self.v = bf16_tensor(b.v_pool)
        self.bt = torch.from_numpy(b.block_table).cuda()
        self.lens = torch.from_numpy(b.kv_lens).cuda()
        self.out = torch.full((b.num_seqs, b.q_len, b.num_q_heads, b.head_dim), float("nan"),
                              dtype=torch.bfloat16, device="cuda")
        self.ws = torch.empty(max(api.attn_workspace_bytes(self.geom), 256), dtype=torch.uint8, device="cuda")

    def status(self) -> int:
        return int(self.ws[:4].view(torch.int32).item())

    def decode(self):
        api.ts_decode_attn(self.geom, self.q, self.k, self.v, self.bt, self.lens, self.out, self.ws)
        torch.cuda.synchronize()
        assert self.status() == 0
        return self.out

    def verify(self):
        api.ts_verify_attn(self.geom, self.q, self.k, self.v, self.bt, self.lens, self.out, self.ws)
        torch.cuda.synchronize()
        assert self.status() == 0
        return self.out

    def splitkv(self, max_splits: int, merge: bool = True):
        b = self.b
        po = torch.full((b.num_seqs, max_splits, b.q_len, b.num_q_heads, b.head_dim), float("nan"),
                        dtype=torch.float32, device="cuda")
        pl = torch.full((b.num_seqs, max_splits, b.q_len, b.num_q_heads), float("nan"),
                        dtype=torch.float32, device="cuda")
        ns = torch.full((b.num_seqs,), -7, dtype=torch.int32, device="cuda")
        ws = torch.empty(max(api.splitkv_workspace_bytes(self.geom), 256), dtype=torch.uint8, device="cuda")
        api.ts_decode_attn_splitkv(self.geom, self.q, self.k, self.v, self.bt, self.lens, max_splits, po, pl, ns, ws)
        torch.cuda.synchronize()
        assert int(ws[:4].view(torch.int32).item()) == 0
        if merge:
            api.ts_lse_merge(self.geom, max_splits, po, pl, ns, self.out)
            torch.cuda.synchronize()
        return po, pl, ns


def errors(gpu_out: torch.Tensor, ref: np.ndarray):
    g = bf16_to_f64(gpu_out).reshape(ref.shape)
    diff = g - ref
    max_abs = float(np.abs(diff).max()) if diff.size else 0.0
    denom = float(np.sqrt((ref * ref).sum()))
    rel_l2 = float(np.sqrt((diff * diff).sum()) / denom) if denom > 0 else float(np.sqrt((diff * diff).sum()))
    return max_abs, rel_l2


def assert_close(gpu_out: torch.Tensor, ref: np.ndarray, what: str = ""):
    g = bf16_to_f64(gpu_out).reshape(ref.shape)
    assert np.isfinite(g).all(), f"{what}: non-finite values in the GPU output"
    max_abs, rel_l2 = errors(gpu_out, ref)
    assert max_abs <= MAX_ABS_TOL and rel_l2 <= REL_L2_TOL, f"{what}: max_abs={max_abs:.3e} rel_l2={rel_l2:.3e}"
    return max_abs, rel_l2
