"""Seeded synthetic weights drawn directly on a CUDA device.

Drawing the 6.6e9 values of the 7B shape on the host takes minutes; torch's device-side Philox generator
produces the same distribution (N(0, weight_std), rounded to bf16; norm gains 1) in a second.  Like the rest
of this package the module only draws data and holds none of the method's arithmetic.
"""
from __future__ import annotations


def device_weights(cfg, seed, device):
    """(layers, glob): lists/dicts of CUDA tensors named as in the weight tables of the C ABI."""
    import torch
    g = torch.Generator(device=device)
    g.manual_seed(seed)
    dt = torch.bfloat16 if cfg.dtype == "bf16" else torch.float32

    def mat(rows, cols):
        return (torch.randn(rows, cols, generator=g, device=device, dtype=torch.float32) * cfg.weight_std).to(dt)
    d, f, hd = cfg.d_model, cfg.d_ff, cfg.n_heads * cfg.head_dim
    kv = getattr(cfg, "n_kv_heads", 0) or cfg.n_heads
    ones = lambda: torch.ones(d, dtype=torch.float32, device=device)
    layers = [{"attn_norm": ones(), "wqkv": mat(hd + 2 * kv * cfg.head_dim, d), "wo": mat(d, hd), "mlp_norm": ones(),
               "w_gate_up": mat(2 * f, d), "w_down": mat(d, f)} for _ in range(cfg.n_layers)]
    glob = {"embed": mat(cfg.vocab, d), "lm_head": mat(cfg.vocab, d), "final_norm": ones()}
    return layers, glob


class HostView:
    """Host-side view of device weights, one layer at a time (float32 numpy), for a CPU consumer that walks
    the layers in order and must not hold all of them at once."""

    def __init__(self, layers):
        self.layers = layers

    def __len__(self):
        return len(self.layers)

    def __getitem__(self, l):
        return {k: v.float().cpu().numpy() for k, v in self.layers[l].items()}
