"""Test infrastructure: plain model of which queries may run while swap-ins are in flight.

Section 4.3, "Asynchronous Swapping-in/out": when the adapter or the cached KV of an arriving query is not in
HBM, its blocks are swapped in and the query waits; queries whose blocks are all resident run meanwhile.  The
model is a dictionary block -> ticket of the copy that fills it; a ticket completes when the test says so.
Only tests use this module; it shares nothing with the GPU library.
"""


class InFlight:
    def __init__(self):
        self.ticket_of = {}          # device block -> ticket of the copy still filling it

    def mark(self, blocks, ticket):
        """The listed blocks are targets of the copies of `ticket`; a block marked again follows the newer copy."""
        for b in blocks:
            self.ticket_of[int(b)] = ticket

    def complete(self, ticket):
        """The copies of `ticket` have landed: its blocks are resident."""
        self.ticket_of = {b: t for b, t in self.ticket_of.items() if t != ticket}

    def ready(self, block_lists):
        """ready[r] is True when no block request r touches is still in flight."""
        return [all(int(b) not in self.ticket_of for b in blocks) for blocks in block_lists]

    def count(self):
        return len(self.ticket_of)
