"""Shared helpers of the GPU parity tests: run the oracle on host copies of the very same tensors and
apply the pass criteria (index sets exact outside the |z| < 1e-3 band; y within relative L2 1e-2 and
max-abs 2e-2 * ||y||_inf -- the tolerance stated for bf16 storage with fp32 accumulation)."""
import numpy as np
import torch

import oracle

REL_L2 = 1e-2
MAX_ABS = 2e-2
BAND = 1e-3


def host(t):
    return None if t is None else t.detach().cpu()


def gate_dict_to_oracle(gate):
    """Oracle-side description of a gate dict of device tensors."""
    if "W_g" in gate:
        return dict(W_g=host(gate["W_g"]))
    return dict(lopa=dict(V=host(gate["V"]), U=host(gate["U"]), g_idx=host(gate.get("g_idx")),
                          g_sign=host(gate.get("g_sign")), gamma=host(gate.get("rms_gain")),
                          use_rmsnorm=gate.get("use_rmsnorm", True), eps=gate.get("rms_eps", 1e-5)))


def run_oracle(x, gate, b_g, W_up, W_down, act, route="sparse", threads=8, act_up=None):
    return oracle.ffn(host(x), host(W_up), host(W_down), act, b_g=host(b_g), route=route,
                      threads=threads, act_up=act_up, **gate_dict_to_oracle(gate))


def assert_y_close(y_gpu, y_ref, rel_l2=REL_L2, max_abs=MAX_ABS, what=""):
    y_gpu = np.asarray(y_gpu.detach().cpu().double().numpy()).reshape(y_ref.shape)
    assert np.isfinite(y_gpu).all(), what
    for b in range(y_ref.shape[0] if y_ref.ndim == 2 else 1):
        g = y_gpu[b] if y_ref.ndim == 2 else y_gpu
        r = y_ref[b] if y_ref.ndim == 2 else y_ref
        norm = np.linalg.norm(r)
        if norm == 0.0:
            assert not g.any(), f"{what}: reference is exactly zero, GPU is not"
            continue
        err_l2 = np.linalg.norm(g - r) / norm
        err_max = np.abs(g - r).max() / np.abs(r).max()
        assert err_l2 <= rel_l2, f"{what} token {b}: relative L2 error {err_l2:.3e} > {rel_l2}"
        assert err_max <= max_abs, f"{what} token {b}: max-abs error {err_max:.3e} x ||y||inf > {max_abs}"


def assert_active_set(idx_gpu, ref, what=""):
    """idx_gpu: ascending int32 tensor from the library; ref: oracle output (z [B,H] or [H])."""
    got = idx_gpu.cpu().numpy()
    assert (np.diff(got) > 0).all(), f"{what}: index list not strictly ascending"
    z = ref["z"] if ref["z"].ndim == 2 else ref["z"][None, :]
    want_mask = (z > 0).any(axis=0)
    got_mask = np.zeros(z.shape[1], bool)
    got_mask[got] = True
    diff = np.nonzero(want_mask != got_mask)[0]
    # a neuron may differ only if some token has it inside the dead band and none fires it clearly
    for j in diff:
        clear = (z[:, j] >= BAND).any()
        inband = (np.abs(z[:, j]) < BAND).any()
        assert inband and not clear, f"{what}: neuron {j} differs, z = {z[:, j]}"
    return len(diff)
