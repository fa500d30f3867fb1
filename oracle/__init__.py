"""CPU oracle of the SSN stage-boundary codec.  Test infrastructure only: nothing on the
product path may import this package."""
