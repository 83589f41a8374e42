"""One FO-SGD round trip when the simulated workers are spread over several GPUs.

Every rank owns M_local workers (ids rank*M_local ...).  Per step a rank
  1. encodes its own workers' gradients                      (fosgd_encode)
  2. decodes and sums its own workers, scaled by lambda/(N sqrt n)   (fosgd_server_aggregate)
  3. all-reduces the partial averages (one fp32 vector of d' entries; the only exchange:
     the server average of eq. (4.1) is a sum, so it splits over ranks)
  4. encodes the average for the downlink with the server's id, identically on every rank
     (fosgd_downlink_encode)
  5. decodes the downlink                                     (fosgd_downlink_decode)
With one rank there is no collective and steps 2 and 4 are one library call.
With `amps` (a DeviceAmplitudes) the amplitudes are measured on the device first
(fosgd_amplitudes) and every call reads them from device memory: no host synchronisation in the
step.  Across ranks the single amplitudes, or the server's per-block table, are MAX all-reduced
(all are increasing in the norms they bound); per-worker block tables stay with their rank.

`codec` is the module that provides the five calls (this package by default); the CPU tests
pass a stand-in so that the rank/worker bookkeeping can be exercised under gloo.
"""
from __future__ import annotations

from dataclasses import dataclass


@dataclass
class RoundTripBuffers:
    bits: object      # [M_local, d'/32] int32
    acc: object       # [d'] fp32
    down: object      # [P, d'/32] int32
    out: object       # [d] fp32
    ws: object        # scratch (uint8) or None
    grads_free: object = None   # round_trip_from_host: event after the last read of the staged gradients
    side_streams: object = None  # round_trip(encode_streams > 1): the streams the encoder's sub-batches run on


@dataclass
class DeviceAmplitudes:
    lam: object            # [1] fp32, or [rows, d' >> b] with per_block
    lam_s: object          # [1] fp32, or [d' >> b]
    ws: object             # scratch for the norm pass (fosgd_workspace_bytes of the amplitude op)
    per_block: bool = False
    alpha: float = 2.0
    alpha_s: float = 2.0


def round_trip(codec, grads, d, buf: RoundTripBuffers, lam, lam_s, seed, step, *, K=1, block_log2=0,
               rank=0, world=1, worker_stride=None, group=None, workers=None, amps=None, encode_streams=1):
    """Enqueue one round trip; returns buf.out (the decoded downlink vector, same on all ranks).

    `encode_streams` > 1 cuts the uplink encoder's workers into that many sub-batches on side streams
    (`buf.ws` must hold all the workers): the memory-bound strided pass of one sub-batch then runs
    beside the issue-bound contiguous pass of another, worth about 4 % of the step on the 2^24
    workload; every worker's bits are the same as with one stream.

    `workers` (default: the rows of `grads`) is the number of workers this rank simulates.  If it
    exceeds the rows held in `grads`, the workers are streamed in chunks of that many rows (worker n
    reads row n mod rows; `buf.bits` needs one chunk of rows only) and the server accumulates chunk
    after chunk into `buf.acc`: the footprint stays bounded whatever the worker count."""
    rows = grads.shape[0]
    M_local = rows if workers is None else workers
    id0 = rank * M_local
    if M_local % rows:
        raise ValueError("the worker count must be a multiple of the resident rows")
    chunks = M_local // rows
    final_down = buf.down if world == 1 else None
    dev_amp = amps is not None
    pb = dev_amp and amps.per_block
    # one amplitude for all workers, one rank, all workers resident: the encoder measures the norms itself
    # (fosgd_encode_measured reads the gradients once where its first pass can carry the sums)
    measured_encode = (dev_amp and not amps.per_block and world == 1 and chunks == 1 and encode_streams <= 1
                       and hasattr(codec, "encode_measured"))
    if dev_amp and not measured_encode:
        # every distinct gradient is a row of `grads` (streamed workers cycle through the rows)
        codec.amplitudes(grads, d, amps.lam, amps.lam_s, alpha=amps.alpha, alpha_s=amps.alpha_s,
                         block_log2=block_log2, per_block=pb, ws=amps.ws, worker_stride=worker_stride)
        if world > 1:
            import torch.distributed as dist
            if not pb:
                dist.all_reduce(amps.lam, op=dist.ReduceOp.MAX, group=group)
            dist.all_reduce(amps.lam_s, op=dist.ReduceOp.MAX, group=group)
    for c in range(chunks):
        first = id0 + c * rows
        last = c == chunks - 1
        flags = (codec.AGG_BEGIN if c == 0 else 0) | (codec.AGG_END if last else 0)
        if encode_streams > 1 and rows >= encode_streams:
            _encode_on_streams(codec, grads, d, buf, lam, seed, step, first, block_log2, worker_stride,
                               amps, encode_streams)
        elif measured_encode:
            codec.encode_measured(grads, d, buf.bits, amps.lam, amps.lam_s, seed, step, alpha=amps.alpha,
                                  alpha_s=amps.alpha_s, worker_id0=first, block_log2=block_log2, ws=buf.ws,
                                  amp_ws=amps.ws, worker_stride=worker_stride)
        elif dev_amp:
            codec.encode_dev(grads, d, buf.bits, amps.lam, seed, step, worker_id0=first, block_log2=block_log2,
                             per_block=pb, ws=buf.ws, worker_stride=worker_stride)
        else:
            codec.encode(grads, d, buf.bits, lam, seed, step, worker_id0=first, block_log2=block_log2, ws=buf.ws,
                         worker_stride=worker_stride)
        if dev_amp:
            codec.server_aggregate_dev(buf.bits, d, buf.acc, amps.lam, seed, step, N_total=M_local * world,
                                       worker_id0=first, flags=flags, lam_s=amps.lam_s, K=K,
                                       down_bits=final_down if last else None, block_log2=block_log2,
                                       per_block=pb, ws=buf.ws)
        else:
            codec.server_aggregate(buf.bits, d, buf.acc, lam, seed, step, N_total=M_local * world, worker_id0=first,
                                   flags=flags, lam_s=lam_s, K=K, down_bits=final_down if last else None,
                                   block_log2=block_log2, ws=buf.ws)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(buf.acc, op=dist.ReduceOp.SUM, group=group)
        if dev_amp:
            codec.downlink_encode(buf.acc, d, buf.down, amps.lam_s, seed, step, K=K, block_log2=block_log2,
                                  per_block=pb, ws=buf.ws)
        else:
            codec.downlink_encode(buf.acc, d, buf.down, lam_s, seed, step, K=K, block_log2=block_log2, ws=buf.ws)
    if dev_amp:
        codec.downlink_decode_dev(buf.down, d, buf.out, amps.lam_s, seed, step, K=K, block_log2=block_log2,
                                  per_block=pb, ws=buf.ws)
    else:
        codec.downlink_decode(buf.down, d, buf.out, lam_s, seed, step, K=K, block_log2=block_log2, ws=buf.ws)
    return buf.out


def _encode_on_streams(codec, grads, d, buf, lam, seed, step, first, block_log2, worker_stride, amps, nstreams):
    """The uplink encoder on `nstreams` side streams, each taking an equal share of the rows and its
    own slice of the scratch buffer; the current stream waits for all of them."""
    import torch
    rows = grads.shape[0]
    if buf.side_streams is None or len(buf.side_streams) != nstreams:
        buf.side_streams = [torch.cuda.Stream() for _ in range(nstreams)]
    cur = torch.cuda.current_stream()
    per = -(-rows // nstreams)
    ws_per = (buf.ws.numel() // rows) & ~15 if buf.ws is not None else 0    # slices stay 16-byte aligned
    need = codec.workspace_bytes(codec.OP_ENCODE, d, block_log2=block_log2)
    if ws_per < need:
        raise ValueError(f"encode_streams needs scratch for every resident row: {need} bytes per row, "
                         f"{ws_per} available")
    for k, s in enumerate(buf.side_streams):
        a, b = k * per, min(rows, (k + 1) * per)
        if a >= b:
            break
        s.wait_stream(cur)
        with torch.cuda.stream(s):
            ws = buf.ws[a * ws_per:b * ws_per] if buf.ws is not None else None
            if amps is not None:
                nb = amps.lam.numel() // rows if amps.per_block else 0
                codec.encode_dev(grads[a:b], d, buf.bits[a:b], amps.lam[a * nb:] if amps.per_block else amps.lam, seed,
                                 step, worker_id0=first + a, block_log2=block_log2, per_block=amps.per_block, ws=ws,
                                 worker_stride=worker_stride)
            else:
                codec.encode(grads[a:b], d, buf.bits[a:b], lam, seed, step, worker_id0=first + a,
                             block_log2=block_log2, ws=ws, worker_stride=worker_stride)
        cur.wait_stream(s)


def round_trip_from_host(codec, host_grads, grads, d, buf: RoundTripBuffers, lam, lam_s, seed, step, *, K=1,
                         block_log2=0, rank=0, world=1, worker_stride=None, group=None, pieces=8, copy_stream=None,
                         host_out=None):
    """The same round trip for gradients that start in pinned host memory (`host_grads`, same shape
    as the device buffer `grads`): the rows cross to the device in `pieces` pieces on `copy_stream`
    while the encoder and the server already work on the pieces that have arrived, so the host link
    and the GPU overlap and only the last piece's compute is exposed; the next call's copies wait
    only for this call's last encode (an event kept in `buf`), not for its server tail, downlink
    and copy back.  The server sums pieces as
    integers, so the result is bit for bit that of `round_trip` on the whole batch.  With `host_out`
    (pinned) the decoded vector is copied back at the end.  Amplitudes are passed by value."""
    import torch
    rows = grads.shape[0]
    id0 = rank * rows
    cur = torch.cuda.current_stream()
    copy_stream = copy_stream if copy_stream is not None else torch.cuda.Stream()
    if buf.grads_free is not None:        # the previous step's encoders may still be reading `grads`
        copy_stream.wait_event(buf.grads_free)
    else:
        copy_stream.wait_stream(cur)
    per = -(-rows // max(1, min(pieces, rows)))
    arrived = []
    with torch.cuda.stream(copy_stream):
        for a in range(0, rows, per):
            b = min(rows, a + per)
            grads[a:b].copy_(host_grads[a:b], non_blocking=True)
            ev = torch.cuda.Event()
            ev.record(copy_stream)
            arrived.append((a, b, ev))
    final_down = buf.down if world == 1 else None
    for a, b, ev in arrived:
        cur.wait_event(ev)
        last = b == rows
        flags = (codec.AGG_BEGIN if a == 0 else 0) | (codec.AGG_END if last else 0)
        codec.encode(grads[a:b], d, buf.bits[a:b], lam, seed, step, worker_id0=id0 + a, block_log2=block_log2,
                     ws=buf.ws, worker_stride=worker_stride)
        if last:
            buf.grads_free = torch.cuda.Event()
            buf.grads_free.record(cur)
        codec.server_aggregate(buf.bits[a:b], d, buf.acc, lam, seed, step, N_total=rows * world, worker_id0=id0 + a,
                               flags=flags, lam_s=lam_s, K=K, down_bits=final_down if last else None,
                               block_log2=block_log2, ws=buf.ws)
    if world > 1:
        import torch.distributed as dist
        dist.all_reduce(buf.acc, op=dist.ReduceOp.SUM, group=group)
        codec.downlink_encode(buf.acc, d, buf.down, lam_s, seed, step, K=K, block_log2=block_log2, ws=buf.ws)
    codec.downlink_decode(buf.down, d, buf.out, lam_s, seed, step, K=K, block_log2=block_log2, ws=buf.ws)
    if host_out is not None:
        host_out.copy_(buf.out, non_blocking=True)
    return buf.out
