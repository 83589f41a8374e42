"""A stand-in for the package's Python binding with the same call signatures, computed by the CPU
oracle on torch CPU tensors: lets the host-side drivers (multi-rank round trip, closed loop) run
without a GPU, and gives the GPU tests a reference trajectory."""
import numpy as np
import torch

import oracle


class OracleCodec:
    """Same call signatures as the package, computed by the CPU oracle on torch CPU tensors."""
    SERVER_ID = oracle.SERVER_ID
    AGG_BEGIN, AGG_END = 1, 2

    @staticmethod
    def encode(grads, d, bits, lam, seed, step, worker_id0=0, block_log2=0, ws=None, worker_stride=None):
        for n in range(grads.shape[0]):
            wid = worker_id0 if worker_id0 == oracle.SERVER_ID else worker_id0 + n
            w = oracle.encode(grads[n, :d].double().numpy(), seed, step, wid, lam, block_log2=block_log2)[0]
            bits.view(-1, bits.shape[-1])[n].copy_(torch.from_numpy(w.view(np.int32)))

    @staticmethod
    def server_aggregate(bits, d, acc, lam, seed, step, N_total=None, worker_id0=0, flags=3, lam_s=0.0, K=1,
                         down_bits=None, block_log2=0, ws=None):
        # the stand-in keeps the running sum in decoded units (the library keeps integers until END)
        M = bits.shape[0]
        N = M if N_total is None else N_total
        g = oracle.aggregate(bits.numpy().view(np.uint32), d, seed, step, lam, worker_id0=worker_id0,
                             block_log2=block_log2) * M
        part = torch.from_numpy(g)
        total = part if flags & 1 else acc.double() + part
        if flags & 2:
            total = total / N
        acc.copy_(total.float())
        if down_bits is not None and flags & 2:
            pl = oracle.downlink_encode(acc.double().numpy(), seed, step, lam_s, K=K, block_log2=block_log2)
            down_bits.copy_(torch.from_numpy(pl.view(np.int32)))

    @staticmethod
    def downlink_decode(down, d, out, lam_s, seed, step, K=1, block_log2=0, ws=None):
        dp = down.shape[-1] * 32
        o = oracle.downlink_decode(down.numpy().view(np.uint32), dp, seed, step, lam_s, K=K, block_log2=block_log2)
        out.copy_(torch.from_numpy(o[:d]).float())


    # amplitudes held in tensors, as the library's *_dev calls read them
    @staticmethod
    def amplitudes(grads, d, lam, lam_s=None, alpha=2.0, alpha_s=2.0, block_log2=0, per_block=False, ws=None,
                   worker_stride=None):
        G = grads[:, :d].double().numpy()
        if per_block:
            t, ts = oracle.block_amplitudes(G, alpha, alpha_s, block_log2)
            lam.copy_(torch.from_numpy(t).float().view(lam.shape))
            lam_s.copy_(torch.from_numpy(ts).float())
            return
        n = oracle.transform_len(d, block_log2)
        l = oracle.lam(float(np.linalg.norm(G, axis=1).max()), alpha, n)
        lam.fill_(l)
        lam_s.fill_(oracle.lam_server(l, alpha_s, n))

    @staticmethod
    def _amp(t, per_block, rows=None):
        if isinstance(t, (int, float)):
            return float(t)
        if not per_block:
            return float(t.view(-1)[0])
        a = t.double().numpy()
        return a.reshape(rows, -1) if rows else a.reshape(-1)

    @classmethod
    def encode_dev(cls, grads, d, bits, lam, seed, step, per_block=False, **kw):
        if not per_block:
            return cls.encode(grads, d, bits, cls._amp(lam, False), seed, step, **kw)
        tab = cls._amp(lam, True, grads.shape[0])
        for n in range(grads.shape[0]):           # one worker at a time, each with its own table row
            wid = kw.get("worker_id0", 0)
            one = dict(kw, worker_id0=wid if wid == oracle.SERVER_ID else wid + n)
            cls.encode(grads[n:n + 1], d, bits.view(-1, bits.shape[-1])[n:n + 1], tab[n], seed, step, **one)

    @classmethod
    def server_aggregate_dev(cls, bits, d, acc, lam, seed, step, lam_s=None, per_block=False, **kw):
        cls.server_aggregate(bits, d, acc, cls._amp(lam, per_block, bits.shape[0]), seed, step,
                             lam_s=None if lam_s is None else cls._amp(lam_s, per_block), **kw)

    @classmethod
    def downlink_decode_dev(cls, down, d, out, lam_s, seed, step, per_block=False, **kw):
        cls.downlink_decode(down, d, out, cls._amp(lam_s, per_block), seed, step, **kw)

    # ---- what closed_loop.run needs besides the calls above ----
    OP_ENCODE, OP_AGGREGATE, OP_AMPLITUDES, OP_BLOCK_AMPLITUDES = 0, 2, 5, 6
    padded_dim = staticmethod(oracle.padded_dim)
    planes = staticmethod(oracle.planes)

    @staticmethod
    def workspace_bytes(op, d, M=1, block_log2=0, K=1):
        return 0

    @classmethod
    def downlink_encode(cls, gbar, d, down, lam_s, seed, step, K=1, block_log2=0, per_block=False, ws=None):
        pl = oracle.downlink_encode(gbar.double().numpy(), seed, step, cls._amp(lam_s, per_block), K=K,
                                    block_log2=block_log2)
        down.copy_(torch.from_numpy(pl.view(np.int32)))

    @classmethod
    def downlink_apply(cls, down, d, x, lam_s, seed, step, step_size, K=1, block_log2=0, per_block=False, ws=None):
        # eq. (4.2): x <- x - delta * g^d
        dp = down.shape[-1] * 32
        g = oracle.downlink_decode(down.numpy().view(np.uint32), dp, seed, step, cls._amp(lam_s, per_block), K=K,
                                   block_log2=block_log2)
        x.copy_((x.double() - step_size * torch.from_numpy(g[:d])).float())
