"""Two caches driven at the same time on two streams. A handle owns everything its kernels use beyond the
caller's buffers (tables, tile lists, the verification's partial sums and ticket), so launches of two
handles may overlap on the GPU in any order: each must end with exactly the bits it produces when it runs
alone. (The one entry point that shares scratch between calls is speca_verify_pred_static; its header
says so and it is not used here.)"""
import pytest
import torch

pytestmark = pytest.mark.gpu

DEV = "cuda:0"


@pytest.fixture(scope="module")
def S():
    from paper_2509_11628_b200 import binding
    binding._lib()
    return binding


def bits(x):
    return x.contiguous().view(torch.uint8)


class Run:
    """One cache and the buffers of its sampler loop; `step(k)` enqueues step k on `stream` without waiting."""

    def __init__(self, S, entries, B, m, layout, seed, stream):
        self.S, self.entries, self.B, self.m, self.stream = S, entries, B, m, stream
        self.cache = S.SpecaCache(entries, B, m, 1, DEV, verify_entry=len(entries) - 1, layout=layout)
        gen = torch.Generator(device=DEV).manual_seed(seed)
        # a smooth path in t plus a little noise, so that some samples accept and some do not
        self.base = [torch.randn(B, n, d, generator=gen, device=DEV) for n, d in entries]
        self.slope = [torch.randn(B, n, d, generator=gen, device=DEV) for n, d in entries]
        self.noise = [torch.randn(B, n, d, generator=gen, device=DEV) for n, d in entries]
        self.scale = torch.tensor([0.002 * (1 + 7 * (b % 3)) for b in range(B)], device=DEV).view(B, 1, 1)
        self.outs = [torch.zeros(B, n, d, dtype=torch.bfloat16, device=DEV) for n, d in entries]
        self.err = torch.zeros(B, dtype=torch.float32, device=DEV)
        self.accept = torch.zeros(B, dtype=torch.uint8, device=DEV)
        self.active = torch.ones(B, dtype=torch.uint8, device=DEV)
        self.nxt = torch.zeros(B, dtype=torch.uint8, device=DEV)
        self.spec = torch.zeros(B, dtype=torch.int32, device=DEV)
        self.log = []

    def feature(self, e, t, k):
        return (self.base[e] + t * self.slope[e] + t * t * 0.5 * self.base[e] +
                self.scale * ((k % 5) - 2) * self.noise[e]).bfloat16()

    def step(self, k):
        t = 1.0 - 0.03 * k
        B, ne = self.B, len(self.entries)
        with torch.cuda.stream(self.stream):
            if k <= self.m or k % 4 == 0:       # reference step, with the next step's forecasts in the same launch
                feats = [self.feature(e, t, k) for e in range(ne)]
                give = list(self.outs)
                give[-1] = None
                self.cache.update_forecast(feats, [t] * B, [t - 0.03] * B, give, active=self.active, spec_count=self.spec,
                                           rearm=self.active, stream=self.stream)
            else:                               # speculative step: the forecasts are there; verify and continue
                fresh = self.feature(ne - 1, t, k)
                self.cache.verify_select(fresh, [t] * B, [0.02] * B, self.err, self.accept, self.active, self.nxt, 3, 1,
                                         self.spec, out_pred=self.outs[-1], stream=self.stream)
                self.active, self.nxt = self.nxt, self.active
                others = list(self.outs)
                others[-1] = None
                self.cache.forecast([t - 0.03] * B, others, self.active, stream=self.stream)
                self.log.append((self.err.clone(), self.accept.clone(), self.active.clone(), self.spec.clone()))
            self.log.append(tuple(o.clone() for o in self.outs))

    def close(self):
        self.cache.close()


def flat(log):
    out = []
    for item in log:
        out.extend(item)
    return out


@pytest.mark.parametrize("layout_a,layout_b", [(0, 0), (0, 1)])
def test_two_handles_on_two_streams_give_the_bits_they_give_alone(S, layout_a, layout_b):
    shape_a = ([(300, 1152), (77, 1031), (512, 1152)], 6, 2)
    shape_b = ([(640, 3072), (1200, 3072)], 2, 3)
    steps = 14
    # alone, one after the other, on the default stream
    alone = []
    for (entries, B, m), layout, seed in ((shape_a, layout_a, 1), (shape_b, layout_b, 2)):
        r = Run(S, entries, B, m, layout, seed, torch.cuda.current_stream(DEV))
        for k in range(steps):
            r.step(k)
        torch.cuda.synchronize()
        alone.append(flat(r.log))
        r.close()
    # together: step k of both enqueued back to back on two streams, nothing waits in between
    s1, s2 = torch.cuda.Stream(DEV), torch.cuda.Stream(DEV)
    torch.cuda.synchronize()
    ra = Run(S, *shape_a, layout_a, 1, s1)
    rb = Run(S, *shape_b, layout_b, 2, s2)
    torch.cuda.synchronize()                    # the set-up ran on the default stream
    for k in range(steps):
        ra.step(k)
        rb.step(k)
    torch.cuda.synchronize()
    for which, (r, ref) in enumerate(((ra, alone[0]), (rb, alone[1]))):
        got = flat(r.log)
        assert len(got) == len(ref)
        for i, (g, w) in enumerate(zip(got, ref)):
            assert torch.equal(bits(g), bits(w)), "handle %d, logged tensor %d" % (which, i)
    decisions = [x for x in flat(ra.log) if x.dtype == torch.uint8 and x.numel() == 6]
    assert any(bool(d.any()) for d in decisions) and any(not bool(d.all()) for d in decisions)   # both outcomes occurred
    ra.close()
    rb.close()
