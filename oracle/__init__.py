"""CPU oracle of the HiSpec verification path. Test infrastructure only: the
product never imports this package."""
