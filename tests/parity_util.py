"""Helpers for the GPU parity tests: run the CUDA path through the C ABI and the
fp64 oracle on the same seeded buffers, and compare.

Decode parity feeds the GPU-built team records into the oracle's Algorithm 1
(which takes team records as an input); team-building parity is tested on its
own against the oracle's Algorithm 2.
"""
import math

import numpy as np
import torch

from oracle import santapp_oracle as orc
from paper_2609_35629_b200 import binding as sp
from paper_2609_35629_b200 import synth


def geometry(spec: synth.WorkloadSpec) -> sp.Geometry:
    return sp.Geometry(spec.n_seqs, spec.n_q_heads, spec.n_kv_heads, spec.head_dim, spec.parent_size,
                       spec.reps_per_parent, sp.SANTAPP_FP16 if spec.elem == "fp16" else sp.SANTAPP_BF16)


class GpuLayer:
    """One layer's buffers on the GPU plus host copies of the team records."""

    def __init__(self, spec, data, device="cuda", builder=None):
        self.spec, self.data = spec, data
        self.geom = geometry(spec)
        self.k_prompt = sp.bf16_bits_to_cuda(data.k_prompt, device, self.geom.torch_dtype)
        self.v_prompt = sp.bf16_bits_to_cuda(data.v_prompt, device, self.geom.torch_dtype)
        self.k_suffix = sp.bf16_bits_to_cuda(data.k_suffix, device, self.geom.torch_dtype)
        self.v_suffix = sp.bf16_bits_to_cuda(data.v_suffix, device, self.geom.torch_dtype)
        self.teams = (builder or sp.santapp_build_teams)(self.geom, spec.prompt_len, self.k_prompt, self.v_prompt)
        torch.cuda.synchronize()
        t = self.teams
        self.team_row_start = t.team_row_start.cpu().numpy()
        self.row_token = t.row_token.cpu().numpy()
        self.rep_bits = t.rep_keys.view(torch.int16).cpu().numpy().view(np.uint16)
        self.k_packed_bits = t.k_packed.view(torch.int16).cpu().numpy().view(np.uint16)
        self.v_packed_bits = t.v_packed.view(torch.int16).cpu().numpy().view(np.uint16)
        self.seq_row_off = t.seq_row_off.cpu().numpy()
        self.seq_team_off = t.seq_team_off.cpu().numpy()
        self.team_count = t.team_count.cpu().numpy()

    def records(self, b, j):
        """(team_start[M+1], team_member[N], rep_key[M, d] fp64) of sequence b, KV head j."""
        t0 = int(self.seq_team_off[b])
        t1 = t0 + int(self.team_count[j, b])          # the pair's teams; later slots of the sequence are empty
        r0, r1 = int(self.seq_row_off[b]), int(self.seq_row_off[b + 1])
        ts = self.team_row_start[j, t0 + b: t1 + b + 1].astype(np.int32)
        tm = self.row_token[j, r0:r1].astype(np.int32)
        rep = synth.to_f64(self.rep_bits[j, t0:t1], self.spec.elem)
        return ts, tm, rep

    def oracle_inputs(self, b):
        """Per-sequence arrays in the oracle's decode_step layout."""
        spec = self.spec
        r0, r1 = int(self.seq_row_off[b]), int(self.seq_row_off[b + 1])
        N = r1 - r0
        recs = [self.records(b, j) for j in range(spec.n_kv_heads)]
        M = np.array([len(r[0]) - 1 for r in recs], dtype=np.int32)
        M_max = int(M.max())
        ts = np.zeros((spec.n_kv_heads, M_max + 1), dtype=np.int32)
        tm = np.zeros((spec.n_kv_heads, N), dtype=np.int32)
        rk = np.zeros((spec.n_kv_heads, M_max, spec.head_dim))
        for j, (s, m, rep) in enumerate(recs):
            ts[j, :len(s)] = s
            tm[j] = m
            rk[j, :len(rep)] = rep
        k = synth.to_f64(self.data.k_prompt[:, r0:r1], self.spec.elem)
        v = synth.to_f64(self.data.v_prompt[:, r0:r1], self.spec.elem)
        return dict(k=k, v=v, M=M, ts=ts, tm=tm, rk=rk, N=N)


def oracle_step(layer: GpuLayer, q_bits, suffix_len, K, seed, step, stream_base=0, n_threads=4, dense=False,
                seqs=None):
    """Oracle result for the listed sequences: dict b -> StepResult (or dense output)."""
    spec = layer.spec
    scale = 1.0 / math.sqrt(spec.head_dim)
    out = {}
    for b in (range(spec.n_seqs) if seqs is None else seqs):
        oi = layer.oracle_inputs(b)
        t = int(suffix_len[b])
        ks = synth.to_f64(layer.data.k_suffix[b, :, :t], spec.elem) if t else None
        vs = synth.to_f64(layer.data.v_suffix[b, :, :t], spec.elem) if t else None
        q = synth.to_f64(q_bits[b], spec.elem)
        if dense:
            out[b] = orc.dense_step(q, oi["k"], oi["v"], ks, vs, scale, n_threads=n_threads)
        else:
            out[b] = orc.decode_step(q, oi["k"], oi["v"], oi["M"], oi["ts"], oi["tm"], oi["rk"], ks, vs, K,
                                     seed, step, stream_base + b, scale, n_threads=n_threads)
    return out


def gpu_step(layer: GpuLayer, q_bits, suffix_len, K, seed, step, stream_base=0, dense=False, debug=True):
    spec = layer.spec
    q = sp.bf16_bits_to_cuda(q_bits, dtype=layer.geom.torch_dtype)
    sl = torch.from_numpy(np.asarray(suffix_len, dtype=np.int32)).cuda()
    if dense:
        out = sp.santapp_dense_decode_attn(layer.geom, layer.teams, q, layer.k_suffix, layer.v_suffix, sl)
        torch.cuda.synchronize()
        return out.cpu().numpy(), None
    dbg = sp.DebugBuffers(layer.geom, K, "cuda") if debug else None
    out = sp.santapp_decode_attn(layer.geom, layer.teams, q, layer.k_suffix, layer.v_suffix, sl, K, seed, step,
                                 stream_base=stream_base, debug=dbg)
    torch.cuda.synchronize()
    return out.cpu().numpy(), dbg


def max_abs_v(layer: GpuLayer):
    return float(np.abs(synth.to_f32(layer.data.v_prompt, layer.spec.elem)).max())


def assert_same_sample(sel_gpu, logc_gpu, sel_ref, logc_ref, what=""):
    """Sampled teams of one head: the same set, the same log c per team, and the same order by
    perturbed score -- except that two neighbours in that order may have changed places (both
    sides sum the fp64 routing dot product in a different order, so a near-tie between two
    SELECTED teams may fall either way; the sample, tau and every correction are the same then)."""
    sel_gpu, sel_ref = np.asarray(sel_gpu), np.asarray(sel_ref)
    assert sorted(sel_gpu.tolist()) == sorted(sel_ref.tolist()), f"sampled teams differ {what}"
    pos = {int(g): i for i, g in enumerate(sel_ref)}
    for i, g in enumerate(sel_gpu):
        assert abs(pos[int(g)] - i) <= 1, f"order of the sample differs by more than a swap of neighbours {what}"
        assert abs(float(logc_gpu[i]) - float(logc_ref[pos[int(g)]])) <= 1e-5, f"log c differs {what}"
