"""Host-side sequencing of one DP-SGD macro-step over the C ABI (no arithmetic here).

Algorithm 1's g_t needs, per microbatch, the per-example norms over ALL layers before any layer can be
scaled, hence two passes over (A, G): norms -> clip factors -> clipped accumulate.  Noise, the division by
the macro-batch size and the AdamW update run once per macro-batch (Section 5.3) as one fused pass.
"""
from __future__ import annotations

from typing import List, Optional, Sequence

import torch

from . import binding as b
from .synth import EMBEDDING, LAYERNORM, LINEAR, LayerData, LayerSpec


class DeviceStatusError(RuntimeError):
    """The library's device-side status word was not clean when a macro-batch was about to be applied."""

    def __init__(self, code: int):
        self.code = int(code)
        try:
            what = b.status_string(self.code)
        except Exception:          # the library itself is missing
            what = "?"
        super().__init__(f"device status {self.code} ({what}): the macro-batch was discarded, "
                         "parameters and optimizer state are unchanged")


class DPStep:
    """Owns the flat fp32 state (theta, m, v, accumulator) for a list of layer specs.

    Tensors are laid end to end in spec order (weight then bias), each start rounded up to a multiple of
    4 elements so that every tensor is 16-byte aligned and one fused launch covers the whole vector.  The
    flat index of an element is also its Philox element index.
    """

    def __init__(self, specs: Sequence[LayerSpec], device, C: float, sigma: float, lr: float, beta1: float,
                 beta2: float, xi: float, weight_decay: float, seed: int = 0, theta: Optional[torch.Tensor] = None,
                 track_snr: bool = False, shared_tables: Optional[dict] = None, shard_world: int = 1):
        """shard_world: number of data-parallel ranks the macro-batch will be finished across (parallel.ShardedUpdate).
        The accumulator and theta are then allocated with room for `shard_world` equal shards (acc_store,
        theta_store; acc and theta are their first n_flat elements), so that the reduce-scatter and the all-gather
        of a macro-batch's end run in place.

        shared_tables maps the index of an output-projection spec (a bias-free LINEAR layer with d_in = V whose
        A is dlogits and whose G is the projection's input) to the index of the EMBEDDING spec whose [V, d] table it
        also trains (BERT's masked-LM decoder): the projection gets no storage of its own, both layers accumulate into
        the table, and the per-example norm includes the inner product of their two contributions."""
        self.specs = list(specs)
        self.shared_tables = dict(shared_tables or {})
        for p_li, e_li in self.shared_tables.items():
            sp, se = self.specs[p_li], self.specs[e_li]
            if not (e_li < p_li and se.kind == EMBEDDING and sp.kind == LINEAR and not sp.has_bias
                    and sp.d_in == se.d_in and sp.d_out == se.d_out):
                raise ValueError("a shared table needs an EMBEDDING [V, d] listed before a bias-free LINEAR V -> d")
        self.device = torch.device(device)
        self.C, self.sigma, self.lr, self.beta1, self.beta2 = C, sigma, lr, beta1, beta2
        self.xi, self.weight_decay, self.seed = xi, weight_decay, seed
        self.offsets: List[List[int]] = []
        self.shapes: List[List[tuple]] = []
        pos = 0
        for li, sp in enumerate(self.specs):
            if li in self.shared_tables:              # alias of the embedding's table
                e_li = self.shared_tables[li]
                self.offsets.append(list(self.offsets[e_li]))
                self.shapes.append(list(self.shapes[e_li]))
                continue
            if sp.kind == LINEAR:
                shp = [(sp.d_in, sp.d_out)] + ([(sp.d_out,)] if sp.has_bias else [])
            elif sp.kind == LAYERNORM:
                shp = [(sp.d_out,), (sp.d_out,)]
            else:
                shp = [(sp.d_in, sp.d_out)]
            offs = []
            for s in shp:
                offs.append(pos)
                n = 1
                for x in s:
                    n *= x
                pos += (n + 3) // 4 * 4
            self.offsets.append(offs)
            self.shapes.append(shp)
        self.n_flat = pos
        from .parallel import padded_length
        cap = padded_length(pos, shard_world)
        self.acc_store = torch.zeros(cap, dtype=torch.float32, device=self.device)
        self.acc = self.acc_store[:pos]
        self.m = torch.zeros(pos, dtype=torch.float32, device=self.device)
        self.v = torch.zeros_like(self.m)
        self.theta_store = torch.zeros_like(self.acc_store) if theta is None else None
        self.theta = self.theta_store[:pos] if theta is None else theta
        self.t = 0
        self.examples_seen = 0
        # gradient-SNR of Section 5.2.1: (sum acc^2, sum noise^2) of the last macro-batch, filled by the fused pass
        self.sq_sums = torch.zeros(2, dtype=torch.float64, device=self.device) if track_snr else None
        self._ws = None
        self._sqnorm = None
        self._clip = None

    def view(self, flat: torch.Tensor, li: int, k: int) -> torch.Tensor:
        shp = self.shapes[li][k]
        n = 1
        for x in shp:
            n *= x
        off = self.offsets[li][k]
        return flat[off:off + n].view(*shp)

    def layer_list(self, data: Sequence[LayerData], paths: Optional[Sequence[int]] = None) -> b.LayerList:
        """Descriptors for one microbatch; data[k] must correspond to specs[k]."""
        out = []
        for li, ld in enumerate(data):
            sp = self.specs[li]
            assert ld.spec.kind == sp.kind and ld.spec.d_out == sp.d_out
            acc_w = self.view(self.acc, li, 0)
            acc_b = self.view(self.acc, li, 1) if len(self.shapes[li]) > 1 else None
            out.append(b.Layer(kind=sp.kind, G=ld.G, A=ld.A, ids=ld.ids, acc_w=acc_w, acc_b=acc_b,
                               has_bias=sp.has_bias, vocab=sp.d_in if sp.kind == EMBEDDING else 0,
                               path=b.DP_PATH_AUTO if paths is None else paths[li]))
        return b.LayerList(out)

    def layer_lists(self, data: Sequence[LayerData], paths: Optional[Sequence[int]] = None) -> List[b.LayerList]:
        """Descriptors for one microbatch whose layers do not all see the same number of tokens (encoder layers per
        token, the masked-LM head per masked position, pooler and sentence classifier per example): one list per
        token count, in order of first appearance; accumulate_microbatch takes the result."""
        whole = self.layer_list(data, paths)
        groups: dict = {}
        for L in whole.layers:
            groups.setdefault(int(L.G.shape[1]), []).append(L)
        return [b.LayerList(ls) for ls in groups.values()]

    def accumulate_microbatch(self, layers, stream=None):
        """norms -> clip factors -> clipped accumulate for one microbatch (all enqueued, no sync).
        `layers` is a LayerList, or a list of them (layer_lists) when token counts differ between layers."""
        lists = [layers] if isinstance(layers, b.LayerList) else list(layers)
        B = lists[0].B
        if self._sqnorm is None or self._sqnorm.numel() != B:
            self._sqnorm = torch.empty(B, dtype=torch.float32, device=self.device)
            self._clip = torch.empty(B, dtype=torch.float32, device=self.device)
        if self._ws is None or len(self._ws) != len(lists):
            self._ws = [None] * len(lists)
        for k, ll in enumerate(lists):
            need = b.dp_workspace_bytes(ll)
            if self._ws[k] is None or self._ws[k].numel() < need:
                self._ws[k] = torch.empty(max(need, 256), dtype=torch.uint8, device=self.device)
            b.dp_per_example_sqnorms(ll, self._sqnorm, k > 0, self._ws[k], stream)
        if self.shared_tables:
            by_acc = {}
            for ll in lists:
                for L in ll.layers:
                    by_acc.setdefault(L.acc_w.data_ptr(), []).append(L)
            for pair in by_acc.values():          # an embedding and the projection that shares its accumulator
                if len(pair) == 2:
                    emb, proj = (pair[0], pair[1]) if pair[0].kind == EMBEDDING else (pair[1], pair[0])
                    b.dp_shared_table_cross_sqnorms(emb, proj, self._sqnorm, stream)
        b.dp_clip_factors(self._sqnorm, self.C, self._clip, stream)
        for k, ll in enumerate(lists):
            b.dp_clipped_accumulate_after_sqnorms(ll, self._clip, self._ws[k], stream)
        self.examples_seen += B
        return self._sqnorm, self._clip

    def discard_macro_batch(self) -> None:
        """Drops the partly accumulated macro-batch: the accumulator is cleared, theta, m, v and t stay as they are."""
        self.acc.zero_()
        self.examples_seen = 0

    def check_device_status(self, stream=None) -> None:
        """Waits for the stream and reads the library's sticky status word.  A bounded wait that ran out or a token
        id out of range makes the kernels skip the offending work, so a squared norm may be wrong and the factor
        min(1, C/||g_i||) would no longer bound that example's contribution by C -- the sensitivity that the noise of
        Algorithm 1 is calibrated to.  In that case the macro-batch is discarded and DeviceStatusError raised."""
        code = b.dp_poll_status(stream)
        if code != b.DP_OK:
            self.discard_macro_batch()
            raise DeviceStatusError(code)

    def finish_macro_batch(self, batch_size: Optional[int] = None, fused: bool = True, stream=None,
                           check_status: bool = True):
        """Noise, division by the macro-batch size and the AdamW update; clears the accumulator.
        With check_status (one host synchronisation per macro-batch) a device-side error reported since the last
        poll raises DeviceStatusError BEFORE anything is applied: theta, m, v and t are untouched and the
        accumulator is cleared."""
        if check_status:
            self.check_device_status(stream)
        N = self.examples_seen if batch_size is None else batch_size
        self.t += 1
        if fused and self.sq_sums is not None:
            self.sq_sums.zero_()
            b.dp_noise_scale_adamw_step_snr(self.theta, self.m, self.v, self.acc, True, self.sigma, self.C, N,
                                            self.seed, self.t, self.lr, self.beta1, self.beta2, self.xi,
                                            self.weight_decay, self.t, self.sq_sums, 0, stream)
        elif fused:
            b.dp_noise_scale_adamw_step(self.theta, self.m, self.v, self.acc, True, self.sigma, self.C, N, self.seed,
                                        self.t, self.lr, self.beta1, self.beta2, self.xi, self.weight_decay, self.t,
                                        0, stream)
        else:
            b.dp_add_noise_and_scale(self.acc, self.sigma, self.C, N, self.seed, self.t, 0, stream)
            b.dp_adamw_step(self.theta, self.m, self.v, self.acc, self.lr, self.beta1, self.beta2, self.xi,
                            self.weight_decay, self.t, stream)
            self.acc.zero_()
        self.examples_seen = 0

    def state_dict(self) -> dict:
        """Everything a run needs to resume in the middle of a macro-batch: parameters, Adam moments, the partly
        filled accumulator, the macro-step counter (which also keys the noise) and the examples seen so far.
        The noise generator is counter-based, so a resumed run draws exactly the noise the original would have."""
        return {"theta": self.theta.clone(), "m": self.m.clone(), "v": self.v.clone(), "acc": self.acc.clone(),
                "t": self.t, "examples_seen": self.examples_seen, "seed": self.seed, "n_flat": self.n_flat}

    def load_state_dict(self, state: dict) -> None:
        if int(state["n_flat"]) != self.n_flat:
            raise ValueError("state belongs to another parameter layout")
        for name in ("theta", "m", "v", "acc"):
            getattr(self, name).copy_(state[name])
        self.t, self.examples_seen, self.seed = int(state["t"]), int(state["examples_seen"]), int(state["seed"])

    def gradient_snr(self) -> float:
        """||aggregated clipped gradient|| / ||noise vector|| of the last finished macro-batch (host sync)."""
        if self.sq_sums is None:
            raise RuntimeError("construct DPStep with track_snr=True")
        s = self.sq_sums.cpu()
        return float((s[0] / s[1]).sqrt()) if float(s[1]) > 0 else float("inf")
