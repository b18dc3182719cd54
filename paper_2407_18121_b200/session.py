"""Buffer management around the C ABI: owns the device tensors and workspaces of one
workload shape and sequences the three calls. No arithmetic happens here.

    s = ElasticCacheSession(N, H, T, D, keep_ratio=0.5, offset=16, scale=1/sqrt(D))
    s.compress(Q, K, V)                  # importance -> select/merge; cache ready, len = budget
    s.compress_with_attention(Q, K, V, out)   # the same, with the prompt's attention output as a by-product
    s.decode(q_all, k_all, v_all, out)   # [steps, N, H, D] each; fixed-point eviction every step

`compress_host` / `decode_host` take pinned host tensors and include the host<->device
copies (on the current stream), for callers whose data starts on the host.
"""
from __future__ import annotations

from typing import Optional

import torch

from . import binding as ec


class ElasticCacheSession:
    def __init__(self, N: int, H: int, T: int, D: int, keep_ratio: float, offset: int, scale: float,
                 population: int = ec.EC_PER_HEAD, protect_ends: bool = True, extra_rows: int = 0,
                 device: Optional[torch.device] = None):
        self.N, self.H, self.T, self.D = N, H, T, D
        self.scale = float(scale)
        self.offset = int(offset)
        self.population = population
        self.protect_ends = protect_ends
        self.n_keep = ec.ec_keep_count(T, keep_ratio)
        if self.n_keep < 1:
            raise ValueError("invalid prompt length or keep ratio")
        self.cap = self.n_keep + extra_rows
        dev = device or torch.device("cuda", torch.cuda.current_device())
        self.device = dev
        bf, f32, i32 = torch.bfloat16, torch.float32, torch.int32
        self.scores = torch.empty((N, H, T), dtype=f32, device=dev)
        self.Kc = torch.empty((N, H, self.cap, D), dtype=bf, device=dev)
        self.Vc = torch.empty_like(self.Kc)
        self.anchor_pos = torch.empty((N, H, self.n_keep), dtype=i32, device=dev)
        self.ws_imp = torch.empty(ec.ec_importance_workspace(N, H, T, D), dtype=torch.uint8, device=dev)
        self.ws_sel = torch.empty(ec.ec_select_merge_workspace(N, H, T, D, self.n_keep, population),
                                  dtype=torch.uint8, device=dev)
        self.cache = ec.ec_cache_init(self.Kc, self.Vc, 0, max(self.n_keep, 2), min(self.offset, max(self.n_keep, 2) - 1))
        self.ws_dec = torch.empty(ec.ec_decode_workspace(self.cache), dtype=torch.uint8, device=dev)
        self._stage = None      # device staging for the *_host calls, allocated on first use
        self._dstage = None
        self._up = None         # side streams of decode_host
        self._down = None

    # ---- device-resident inputs ------------------------------------------------------
    def compress(self, Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor) -> None:
        """Prompt call: importance, anchor selection and merge. Resets the cache to `n_keep` rows."""
        ec.ec_importance(Q, K, self.scores, None, self.scale, self.ws_imp)
        ec.ec_select_merge(K, V, self.scores, self.n_keep, self.population, self.protect_ends,
                           self.Kc, self.Vc, self.anchor_pos, None, self.ws_sel)
        self.cache = ec.ec_cache_init(self.Kc, self.Vc, self.n_keep, max(self.n_keep, 2),
                                      min(self.offset, max(self.n_keep, 2) - 1))

    def compress_with_attention(self, Q: torch.Tensor, K: torch.Tensor, V: torch.Tensor, out: torch.Tensor,
                                lse: Optional[torch.Tensor] = None) -> None:
        """compress() for callers that also want the prompt's attention output (the model's own forward
        pass): `out` [N,H,T,D] and optionally `lse` [N,H,T] come from ec_prefill_attention, whose
        normaliser also gives the importance by the column-sum pass alone. Same cache afterwards."""
        ec.ec_prefill_attention(Q, K, V, out, lse, self.scores, self.scale, self.ws_imp)
        ec.ec_select_merge(K, V, self.scores, self.n_keep, self.population, self.protect_ends,
                           self.Kc, self.Vc, self.anchor_pos, None, self.ws_sel)
        self.cache = ec.ec_cache_init(self.Kc, self.Vc, self.n_keep, max(self.n_keep, 2),
                                      min(self.offset, max(self.n_keep, 2) - 1))

    def decode(self, q: torch.Tensor, k_new: torch.Tensor, v_new: torch.Tensor, out: torch.Tensor,
               want_slots: bool = False):
        """Generation calls for q, k_new, v_new, out of shape [steps, N, H, D]."""
        return ec.ec_decode_steps(q, k_new, v_new, self.cache, self.scale, out, self.ws_dec, want_slots)

    # ---- a new instruction on top of the current cache ---------------------------------
    def logical_slots(self):
        """Physical slots of the cache rows in queue order (oldest first). Fixed budget: the rows
        before the ring never move; the ring holds the `offset` newest rows, oldest at `ring_head`.
        Retention ratio: the list the library maintains (ec_cache_track_order)."""
        c = self.cache
        if c.policy != 0:
            if not c.queue_slots_host:
                raise ValueError("this retention-ratio cache does not track its queue order")
            return [c.queue_slots_host[j] for j in range(c.len)]
        if c.len < c.budget:
            return list(range(c.len))
        base = c.budget - c.offset
        return list(range(base)) + [base + (c.ring_head + i) % c.offset for i in range(c.offset)]

    def recompress(self, Q_new: torch.Tensor, K_new: torch.Tensor, V_new: torch.Tensor, keep_ratio: float):
        """Encode a new instruction of Tq tokens on top of the cache: importance of the cached rows and
        the new rows under the new tokens' queries, then selection and merge over the concatenation.
        Returns a new session holding the compacted result (this one is left untouched)."""
        N, H, Tq, D = Q_new.shape
        P = self.cache.len
        K_all = torch.empty((N, H, P + Tq, D), dtype=torch.bfloat16, device=self.device)
        V_all = torch.empty_like(K_all)
        ec.ec_cache_concat(self.cache, K_new, V_new, K_all, V_all)
        nxt = ElasticCacheSession(N, H, P + Tq, D, keep_ratio, self.offset, self.scale, self.population,
                                  self.protect_ends, device=self.device)
        ws = torch.empty(ec.ec_importance_workspace(N, H, Tq, D), dtype=torch.uint8, device=self.device)
        ec.ec_importance_prefix(Q_new, K_all, nxt.scores, None, self.scale, ws)
        ec.ec_select_merge(K_all, V_all, nxt.scores, nxt.n_keep, nxt.population, nxt.protect_ends,
                           nxt.Kc, nxt.Vc, nxt.anchor_pos, None, nxt.ws_sel)
        nxt.cache = ec.ec_cache_init(nxt.Kc, nxt.Vc, nxt.n_keep, max(nxt.n_keep, 2),
                                     min(nxt.offset, max(nxt.n_keep, 2) - 1))
        return nxt

    # ---- host-resident inputs --------------------------------------------------------
    def _prompt_staging(self):
        if self._stage is None:
            shp = (self.N, self.H, self.T, self.D)
            self._stage = tuple(torch.empty(shp, dtype=torch.bfloat16, device=self.device) for _ in range(3))
        return self._stage

    def _decode_staging(self, steps: int):
        if self._dstage is None or self._dstage[0].shape[0] < steps:
            shp = (steps, self.N, self.H, self.D)
            self._dstage = tuple(torch.empty(shp, dtype=torch.bfloat16, device=self.device) for _ in range(4))
        return self._dstage

    def compress_host(self, Q_host: torch.Tensor, K_host: torch.Tensor, V_host: torch.Tensor,
                      anchor_pos_host: Optional[torch.Tensor] = None) -> int:
        """compress() from pinned host tensors (ec_compress_host). Returns the bytes copied host->device."""
        Q, K, V = self._prompt_staging()
        ec.ec_compress_host(Q_host, K_host, V_host, Q, K, V, self.scores, self.scale, self.n_keep, self.population,
                            self.protect_ends, self.Kc, self.Vc, self.anchor_pos, anchor_pos_host, self.ws_imp,
                            self.ws_sel)
        self.cache = ec.ec_cache_init(self.Kc, self.Vc, self.n_keep, max(self.n_keep, 2),
                                      min(self.offset, max(self.n_keep, 2) - 1))
        return 3 * Q_host.numel() * Q_host.element_size()

    def decode_host(self, q_host: torch.Tensor, k_host: torch.Tensor, v_host: torch.Tensor,
                    out_host: torch.Tensor, chunk: int = 64):
        """decode() from pinned host tensors [steps, N, H, D] (ec_decode_steps_host); writes out_host.
        Returns (h2d, d2h) bytes. Uploads of later chunks and downloads of finished chunks run on two
        side streams while the current chunk decodes."""
        steps = q_host.shape[0]
        chunk = max(chunk, -(-steps // 31))                 # the native call takes at most 31 chunks
        q, k, v, out = (t[:steps] for t in self._decode_staging(steps))
        if self._up is None:
            self._up, self._down = torch.cuda.Stream(), torch.cuda.Stream()
        ec.ec_decode_steps_host(q_host, k_host, v_host, out_host, q, k, v, out, self.cache, self.scale, self.ws_dec,
                                self._up, self._down, chunk)
        nb = q_host.numel() * q_host.element_size()
        return 3 * nb, nb
